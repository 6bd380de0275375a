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
// and the backward kernel (level_bwd) applies the chain rule to exactly these products, level by level.  Run products are stored as bf16
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

// ---------------------------------------------------------------------------------------------- dyadic forward, fused
// Two or three consecutive levels in one launch (p.fuse): a CTA takes 2^fuse neighbouring products of level p.l and
// builds the whole tree above them,
//     A_k = Dy[l][2k+1] Dy[l][2k]  (k < 2^(fuse-1)),    B_k = A_{2k+1} A_{2k},    C = B_1 B_0,
// writing every product to global memory as it appears and keeping it in shared memory as the next product's operand,
// so the intermediate levels are read back by nobody and the launches (and their tails) between the levels are gone.
// Six tile slots: a product's result replaces the tiles of its own left factor; B_0 waits in tensor memory (columns
// 128..255) while A_2, A_3 and B_1 are made.  grid.x = S * groups, groups = ceil(cnt(l + 1) / 2^(fuse-1)).
template <int HD>
__global__ void __launch_bounds__(256, 1) dyadic_fused_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<256>(c, smem_raw, 6 * kTileB);
    const int half_w = 1 << (p.fuse - 1);                        // A products per group
    const int groups = (p.lv.dy_cnt[p.l + 1] + half_w - 1) / half_w;
    const int s = blockIdx.x / groups, g = blockIdx.x % groups;
    uint8_t* sm = c.smem;
    auto mat = [&](int lvl, int idx) { return p.lv.dy_off[lvl] / (HD * HD) + (long)s * p.lv.dy_cnt[lvl] + idx; };
    // acc(col) = left (slots a, a + 1) x right (slots b, b + 1), the lo x lo term left out
    auto product = [&](uint32_t col, int a, int b) {
        publish();   // operands written by this CTA's threads are visible, and nobody still reads the accumulator
        if (c.tid == 0 && c.ok) {
            tc_fence_after_sync();
            const uint32_t base = smem_u32(sm);
            mma(c.tmem + col, base + a * kTileB, OP_K, base + b * kTileB, OP_MN, HD / 16, HD, false);
            mma(c.tmem + col, base + a * kTileB, OP_K, base + (b + 1) * kTileB, OP_MN, HD / 16, HD, true);
            mma(c.tmem + col, base + (a + 1) * kTileB, OP_K, base + b * kTileB, OP_MN, HD / 16, HD, true);
            umma_commit(&c.bars[1]);
        }
        mma_wait(c);
    };
    // accumulator -> bf16 pair: to global memory as Dy[lvl][idx] (if to_global) and / or into slots a, a + 1 (a >= 0)
    auto readout = [&](uint32_t col, int lvl, int idx, bool to_global, int a) {
        if (!c.ok) return;
        float v[32], hi[32];
        for (int i = 0; i < HD / 64; ++i) {
            const int c0 = c.half * (HD / 2) + i * 32;
            tmem_row32(c.tl + col + c0, v);
#pragma unroll
            for (int x = 0; x < 32; ++x) {
                hi[x] = __bfloat162float(__float2bfloat16_rn(v[x]));
                v[x] -= hi[x];
            }
            if (a >= 0) {
                tile_store32(sm + a * kTileB, c.row, c0, hi);
                tile_store32(sm + (a + 1) * kTileB, c.row, c0, v);
            }
            if (to_global) {
                const size_t o = ((size_t)mat(lvl, idx) * HD + c.row) * HD + c0;
                gstore_bf16x32(p.dyh + o, hi, c.row < HD);
                gstore_bf16x32(p.dyl + o, v, c.row < HD);
            }
        }
    };
    const int l = p.l;
    const int a0 = g * half_w;                                   // first A product of this group (index at level l + 1)
    const int cntA = p.lv.dy_cnt[l + 1], cntB = p.lv.dy_cnt[l + 2], cntC = p.fuse >= 3 ? p.lv.dy_cnt[l + 3] : 0;
    const bool hasA1 = a0 + 1 < cntA, hasB0 = (a0 >> 1) < cntB;
    const bool more = p.fuse >= 3 && hasB0 && a0 + 2 < cntA;     // is there a second half of the tree?
    const bool hasA3 = more && a0 + 3 < cntA, hasB1 = more && (a0 >> 1) + 1 < cntB, hasC = hasB1 && (a0 >> 2) < cntC;
    // The operands of A_k (level-l pair 2k+1, 2k) are requested as soon as their slots are free, on a barrier of their
    // own per parity of k: left factor into slots a, a + 1, right factor into b, b + 1.
    uint64_t* lbar[2] = {&c.bars[0], c.bars + 4};
    uint32_t lph[2] = {0, 0};
    if (c.tid == 0) {
        mbar_init(lbar[1], 1);
        mbar_fence_init();
    }
    __syncthreads();
    // part 1 announces all four tiles and fetches the right factor, part 2 the left one (its slots free up later)
    auto request_a1 = [&](int k, int b_) {
        if (c.tid != 0) return;
        mbar_expect_tx(lbar[k & 1], 4 * kT * HD * 2);
        tma_tile(sm + b_ * kTileB, &tm.dyh, lbar[k & 1], HD, (int)(mat(l, 2 * (a0 + k)) * HD));
        tma_tile(sm + (b_ + 1) * kTileB, &tm.dyl, lbar[k & 1], HD, (int)(mat(l, 2 * (a0 + k)) * HD));
    };
    auto request_a2 = [&](int k, int a) {
        if (c.tid != 0) return;
        tma_tile(sm + a * kTileB, &tm.dyh, lbar[k & 1], HD, (int)(mat(l, 2 * (a0 + k) + 1) * HD));
        tma_tile(sm + (a + 1) * kTileB, &tm.dyl, lbar[k & 1], HD, (int)(mat(l, 2 * (a0 + k) + 1) * HD));
    };
    auto wait_a = [&](int k) {
        if (!mbar_wait(lbar[k & 1], lph[k & 1], c.abort_flag, ST_LEVELS)) c.ok = false;
        lph[k & 1] ^= 1;
    };
    request_a1(0, 2);
    request_a2(0, 0);
    if (hasA1) request_a1(1, 4);                                 // slots 4, 5 are free from the start
    wait_a(0);
    product(0, 0, 2);                                            // A_0
    if (hasA1) request_a2(1, 2);                                 // slots 2, 3 are free again
    readout(0, l + 1, a0, true, 0);                              // A_0 -> slots 0, 1
    if (hasA1) {
        wait_a(1);
        product(0, 2, 4);                                        // A_1
        readout(0, l + 1, a0 + 1, true, 2);                      // -> slots 2, 3
    }
    if (hasB0) {
        product(more ? 128 : 0, 2, 0);                           // B_0 = A_1 A_0; it waits in columns 128.. if there is more
        if (more) {                                              // every slot is free now
            request_a1(2, 2);
            request_a2(2, 0);
        }
        if (hasA3) request_a1(3, 4);
        readout(more ? 128 : 0, l + 2, a0 >> 1, true, -1);
        if (more) {
            wait_a(2);
            product(0, 0, 2);                                    // A_2
            if (hasA3) request_a2(3, 2);
            readout(0, l + 1, a0 + 2, true, 0);                  // -> slots 0, 1
            if (hasA3) {
                wait_a(3);
                product(0, 2, 4);                                // A_3
                readout(0, l + 1, a0 + 3, true, 2);              // -> slots 2, 3
            }
            if (hasB1) {
                product(0, 2, 0);                                // B_1 = A_3 A_2
                readout(0, l + 2, (a0 >> 1) + 1, true, 0);       // -> slots 0, 1 (A_2 has been read)
                if (hasC) {
                    readout(128, 0, 0, false, 4);                // B_0 from its columns -> slots 4, 5
                    product(0, 0, 4);                            // C = B_1 B_0
                    readout(0, l + 3, a0 >> 2, true, -1);
                }
            }
        }
    }
    teardown<256>(c, p.status);
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
    // levels to build: all of them, or for a gated problem up to the highest one a kept chunk pair uses (see level_bwd)
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
        const long row_dst = is_key ? kver_row(p.vl, s, l2, ch) : qver_row(p.vl, s, l2, ch);
        if (c.tid == 0) {
            mbar_expect_tx(&c.bars[0], (first ? 3 : 2) * kT * HD * 2);
            if (first) {
                const long row_src = is_key ? kver_row(p.vl, s, l1, ch) : qver_row(p.vl, s, l1, ch);
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

// ---------------------------------------------------------------------------------------------- level backward
// Chain rule of the version chains and of the run products, one launch per level l1 = nlev-2, ..., 0 (p.l = l1),
// grid.x = S * cnt(l1).  A CTA owns ONE run product Dy[l1][b] and gathers its whole gradient in tensor memory, so nothing
// is added atomically and nothing has to be cleared beforehand:
//   (1) the level above (Dy[l1+1][b'] = Dy[l1][2b'+1] Dy[l1][2b'], finished by the previous launch), dC = dDy[l1+1][b >> 1]:
//         b odd:  dDy = dC Dy[l1][b-1]^T          b even:  dDy = Dy[l1][b+1]^T dC
//   (2) every version step that multiplies by Dy[l1][b]: the 2^l1 chunks ch of one aligned run, all at the same
//       target level l2 > l1, with g = dXv[l2][ch] (what the sweeps wrote there plus what earlier launches added):
//         queries (b even, b >= 2, ch = (b << l1) + 2^l1 + x):   dDy += Qv[l1][ch]^T g,   dQv[l1][ch] += g Dy^T
//         keys    (b odd,          ch = ((b-1) << l1) + x):      dDy += g^T Kv[l1][ch],   dKv[l1][ch] += g Dy
//       (the second product is the chain's carry: added in place to the gradient the sweep left at level l1, which the
//       launch of level l1's own source level, or the chunk chain rule for plane 0, reads next).
// The run products enter as single bf16 operands (their hi plane), like every other operand of a gradient product.
// dDy is written once, as bf16: it is only ever read as an MMA operand (by the next launch and, at level 0, by the
// chunk chain rule as dP).  Runs with b = 0 multiply nothing (no boundary lies before chunk 0): only level 0 writes them.
template <int HD>
__global__ void __launch_bounds__(256, 1) level_bwd_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    const int l1 = p.l, cnt = p.lv.dy_cnt[l1];
    const int s = blockIdx.x / cnt, b = blockIdx.x % cnt;
    const long mat = p.lv.dy_off[l1] / (HD * HD) + (long)s * cnt + b;
    const int is_key = b & 1;
    // the chunks of this run's version steps and their common target level
    const int c0 = is_key ? ((b - 1) << l1) : ((b << l1) + (1 << l1));
    int l2 = 0;
    bool role = is_key || b >= 2;
    if (role) {
        if (!is_key) l2 = lowest_set((unsigned)(b << l1));
        else l2 = l1 + 1 + lowest_set(~((unsigned)c0 >> (l1 + 1)));
        role = l2 < p.nlev;
    }
    int src = 0;
    auto valid = [&](int ch) {   // does chunk ch take the step l1 -> l2 through this run product?
        if (!role || ch >= p.N) return false;
        int l1x, bx;
        if (!version_step(is_key, ch, l2, p.N, l1x, bx, src) || l1x != l1) return false;
        return l2 <= highest_level_reached(p, is_key, s, ch);   // block skipping: levels the sweeps did not reach hold nothing
    };
    auto next_chunk = [&](int from) {
        for (int ch = from; ch < c0 + (1 << l1); ++ch)
            if (valid(ch)) return ch;
        return -1;
    };
    const bool parent = l1 + 1 <= p.nlev - 2 && (b >> 1) >= 1 && (b >> 1) < p.lv.dy_cnt[l1 + 1];
    int ch = next_chunk(c0);
    __nv_bfloat16* out = p.ddy16 + (size_t)mat * HD * HD;
    if (ch < 0 && !parent) {   // nothing multiplies by this run product
        if (b >= 1 || l1 == 0)
            for (int i = threadIdx.x; i < HD * HD / 8; i += 256) reinterpret_cast<uint4*>(out)[i] = make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    __nv_bfloat16* dxv = is_key ? p.dkv : p.dqv;
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<256>(c, smem_raw, 7 * kTileB);
    uint8_t* sm = c.smem;   // slots: 0 Dy, 1 dC, 2 the other factor of the level above, (3, 4) and (5, 6): g and Xv[l1] of a chunk
    constexpr uint32_t colCarry = 0, colAcc = 128;
    auto ver_row = [&](int lvl, int chx) { return is_key ? kver_row(p.vl, s, lvl, chx) : qver_row(p.vl, s, lvl, chx); };
    auto chunk_loads = [&](int chx, int buf) {
        uint8_t* base = sm + (3 + 2 * buf) * kTileB;
        const CUtensorMap* gm = is_key ? &tm.dkv : &tm.dqv;
        const CUtensorMap* xm = is_key ? &tm.kv : &tm.qv;
        tma_tile(base, gm, &c.bars[0], HD, (int)ver_row(l2, chx));
        tma_tile(base + kTileB, xm, &c.bars[0], HD, (int)ver_row(l1, chx));
    };
    if (c.tid == 0) {   // first group: the run product itself, the operands of the level above, the first chunk
        const uint32_t tile = kT * HD * 2;
        mbar_expect_tx(&c.bars[0], (ch >= 0 ? 3 : 0) * tile + (parent ? 2 : 0) * tile);
        if (ch >= 0) {
            tma_tile(sm, &tm.dyh, &c.bars[0], HD, (int)(mat * HD));
            chunk_loads(ch, 0);
        }
        if (parent) {
            const long up = p.lv.dy_off[l1 + 1] / (HD * HD) + (long)s * p.lv.dy_cnt[l1 + 1] + (b >> 1);
            tma_tile(sm + kTileB, &tm.ddy, &c.bars[0], HD, (int)(up * HD));
            tma_tile(sm + 2 * kTileB, &tm.dyh, &c.bars[0], HD, (int)((mat + (is_key ? -1 : 1)) * HD));
        }
    }
    constexpr int NI = HD / 64;
    uint32_t pend[NI][2][8];   // the gradient stored at level l1 for the current chunk (32 bf16 = 64 bytes per piece)
    auto request = [&](long row0) {
#pragma unroll
        for (int i = 0; i < NI; ++i) {
            const __nv_bfloat16* g = dxv + ((size_t)row0 + c.row) * HD + c.half * (HD / 2) + i * 32;
            ld_global_v8(g, pend[i][0]);
            ld_global_v8(g + 16, pend[i][1]);
        }
    };
    auto issue_parent = [&](uint32_t a) {
        if (is_key) mma(c.tmem + colAcc, a + kTileB, OP_K, a + 2 * kTileB, OP_K, HD / 16, HD, false);      // dC B^T
        else        mma(c.tmem + colAcc, a + 2 * kTileB, OP_MN, a + kTileB, OP_MN, HD / 16, HD, false);   // A^T dC
    };
    int buf = 0;
    bool first = true;
#pragma unroll 1
    while (ch >= 0 && c.ok) {
        const long row_lo = ver_row(l1, ch);
        request(row_lo);
        const int nxt = next_chunk(ch + 1);
        loads_wait(c);
        // every thread has read the previous chunk's carry out of tensor memory before the next product overwrites it
        tc_fence_before_sync();
        __syncthreads();
        if (c.tid == 0 && c.ok) {
            if (nxt >= 0) {   // the other buffer's products retired before the previous mma_wait returned
                mbar_expect_tx(&c.bars[0], 2 * kT * HD * 2);
                chunk_loads(nxt, buf ^ 1);
            }
            tc_fence_after_sync();
            const uint32_t a = smem_u32(sm), g = a + (3 + 2 * buf) * kTileB, x = g + kTileB;
            if (first && parent) issue_parent(a);
            const bool acc = !first || parent;
            if (!is_key) {
                mma(c.tmem + colCarry, g, OP_K, a, OP_K, HD / 16, HD, false);     // g Dy^T
                mma(c.tmem + colAcc, x, OP_MN, g, OP_MN, 8, HD, acc);             // Xv^T g
            } else {
                mma(c.tmem + colCarry, g, OP_K, a, OP_MN, HD / 16, HD, false);    // g Dy
                mma(c.tmem + colAcc, g, OP_MN, x, OP_MN, 8, HD, acc);             // g^T Xv
            }
            umma_commit(&c.bars[1]);
        }
        mma_wait(c);
        if (c.ok) {
            float v[32], a[32];
#pragma unroll
            for (int i = 0; i < NI; ++i) {
                const int col = c.half * (HD / 2) + i * 32;
#pragma unroll
                for (int x = 0; x < 16; ++x) {
                    const uint32_t w = pend[i][x >> 3][x & 7];
                    v[2 * x] = __uint_as_float(w << 16);
                    v[2 * x + 1] = __uint_as_float(w & 0xffff0000u);
                }
                tmem_row32(c.tl + colCarry + col, a);
#pragma unroll
                for (int x = 0; x < 32; ++x) v[x] += a[x];
                gstore_bf16x32(dxv + ((size_t)row_lo + c.row) * HD + col, v);
            }
        }
        first = false;
        ch = nxt;
        buf ^= 1;
    }
    if (first && c.ok) {   // no version step: the level above is the only contribution
        loads_wait(c);
        if (c.tid == 0 && c.ok) {
            tc_fence_after_sync();
            issue_parent(smem_u32(sm));
            umma_commit(&c.bars[1]);
        }
        mma_wait(c);
    }
    if (c.ok) {
        float v[32];
        for (int i = 0; i < NI; ++i) {
            const int col = c.half * (HD / 2) + i * 32;
            tmem_row32(c.tl + colAcc + col, v);
            gstore_bf16x32(out + (size_t)c.row * HD + col, v, c.row < HD);
        }
    }
    teardown<256>(c, p.status);
}

// ---------------------------------------------------------------------------------------------- tiles moved to a segment's edge
// grid = (S, d / 64).  Paper Sec. 3.4: after L tokens the cached key of position j is H_{L-1} ... H_{j+1} k_j.  In chunk
// form that is  kc_J = Kright_J R_J  with  R_J = P_{J+1}^T ... P_{N-1}^T,  so a CTA walks the chunks of its slice from the
// last to the first carrying R (bf16 hi + lo in shared memory):  kc_J = Kright_J R,  R <- P_J^T R.
// Both products act on the columns of R independently, so a CTA carries only 64 columns of R (and writes those columns
// of the result): at d = 128 two CTAs share a slice (four with 32 columns each were no faster per step and, at 4096
// tokens, more CTAs than SMs).
// QUERY = true is the mirror image for the context-parallel path (paper Sec. 3.5): the queries pulled back to the start of
// the segment,  x_I = Qleft_I R_I  with  R_I = P_{I-1} ... P_0,  walking the chunks upwards with  R <- P_I R;  the last R is
// the product of the whole segment, which the segment hands to the devices holding later queries.
// Results leave as float32 rows (p.kc, the decoding cache) and / or bf16 rows (p.edge16).
template <int HD, bool QUERY>
__global__ void __launch_bounds__(256, 1) key_cache_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<256>(c, smem_raw, kBar5);
    constexpr int NC = 64;                      // columns of R per CTA
    const int s = blockIdx.x, col0 = blockIdx.y * NC;
    uint8_t* sm = c.smem;   // slots: 0 Kright_J / Qleft_I, 1 P hi, 2 P lo, 3 R hi, 4 R lo ([d x 64] in the first panel)
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
        tma_tile(sm, QUERY ? &tm.qv : &tm.kv, &c.bars[0], HD, (int)((long)s * p.Lp + (long)J * kT));   // version slot 0
        tma_tile(sm + kTileB, &tm.dyh, &c.bars[0], HD, (int)(mat * HD));
        tma_tile(sm + 2 * kTileB, &tm.dyl, &c.bars[0], HD, (int)(mat * HD));
    };
    // Segments (key side, p.nseg > 1): blockIdx.z walks only the chunks [z * seg_chunks, (z+1) * seg_chunks) and leaves its keys
    // advanced to the end of THAT range (bf16, p.edge16) together with the range's product (p.pseg); a second pass
    // (suffix_kernel, apply_product_kernel) carries them on to the end of the sequence.  The walk itself is a serial
    // chain of dependent products, so this is what lets a long prompt use all SMs.
    const int c_lo = p.nseg > 1 ? (int)blockIdx.z * p.seg_chunks : 0;
    const int c_hi = p.nseg > 1 ? min(p.N, c_lo + p.seg_chunks) : p.N, cnt = c_hi - c_lo;
    const int first = QUERY ? c_lo : c_hi - 1, step = QUERY ? 1 : -1;
    if (cnt <= 0) { teardown<256>(c, p.status); return; }
    if (c.tid == 0) issue(first);
#pragma unroll 1
    for (int n = 0, J = first; n < cnt && c.ok; ++n, J += step) {
        const bool more = n + 1 < cnt;
        // the query side also wants the product of the whole segment; so does every key range but the first
        const bool update = QUERY || more || (p.nseg > 1 && blockIdx.z > 0);
        loads_wait(c);
        publish();
        if (c.tid == 0 && c.ok) {
            tc_fence_after_sync();
            const uint32_t a = smem_u32(sm);
            mma(c.tmem, a, OP_K, a + 3 * kTileB, OP_MN, HD / 16, NC, false);                       // X R
            mma(c.tmem, a, OP_K, a + 4 * kTileB, OP_MN, HD / 16, NC, true);
            if (update) {
                constexpr int pop = QUERY ? OP_K : OP_MN;                                          // P R  /  P^T R
                mma(c.tmem + 128, a + 1 * kTileB, pop, a + 3 * kTileB, OP_MN, HD / 16, NC, false);
                mma(c.tmem + 128, a + 2 * kTileB, pop, a + 3 * kTileB, OP_MN, HD / 16, NC, true);
                mma(c.tmem + 128, a + 1 * kTileB, pop, a + 4 * kTileB, OP_MN, HD / 16, NC, true);
            }
            umma_commit(&c.bars[1]);
        }
        mma_wait(c);
        if (!c.ok) break;
        if (c.tid == 0 && more) issue(J + step);   // every product has retired: the operand slots are free again
        const int pos = J * kT + c.row, c0 = c.half * 32;
        float v[32];
        uint32_t hi[16], lo[16];
        tmem_row32(c.tl + c0, v);
        if (p.kc) gstore_f32x32(p.kc + ((size_t)s * p.cap + pos) * HD + col0 + c0, v, pos < p.L);
        if (p.edge16) gstore_bf16x32(p.edge16 + ((size_t)s * p.L + pos) * HD + col0 + c0, v, pos < p.L);
        if (update) {
            tmem_row32(c.tl + 128 + c0, v);
            split32(v, hi, lo);
            if (c.row < HD) {
                tile_store_w16(sm + 3 * kTileB, c.row, c0, hi);
                tile_store_w16(sm + 4 * kTileB, c.row, c0, lo);
            }
            if (!more && p.pseg) {   // the range's product, [S][nseg][2 (hi, lo)][d][d]
                const size_t mi = (size_t)s * (p.nseg > 1 ? p.nseg : 1) + (p.nseg > 1 ? blockIdx.z : 0);
                gstore_bf16_w16(p.pseg + ((mi * 2 + 0) * HD + c.row) * HD + col0 + c0, hi, c.row < HD);
                gstore_bf16_w16(p.pseg + ((mi * 2 + 1) * HD + c.row) * HD + col0 + c0, lo, c.row < HD);
            }
        }
    }
    teardown<256>(c, p.status);
}

// ---------------------------------------------------------------------------------------------- products of key ranges towards the end
// grid = (S, d / 64).  With M_g = the product of key range g (p.pseg, [S][nseg][2][d][d]):  Sfx_{nseg-1} = I,
// Sfx_g = M_{g+1} Sfx_{g+1}  (p.sfx, same layout): what a key advanced to the end of range g still has to be multiplied
// by to reach the end of the sequence.  nseg - 1 dependent products of 64 columns each.
template <int HD>
__global__ void __launch_bounds__(256, 1) suffix_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<128>(c, smem_raw, kBar4);
    constexpr int NC = 64;
    const int s = blockIdx.x, col0 = blockIdx.y * NC, c0 = c.half * 32;
    uint8_t* sm = c.smem;   // slots: 0 M hi, 1 M lo, 2 R hi, 3 R lo
    for (int i = c.tid; i < (int)(4 * kTileB / 16); i += 256) reinterpret_cast<uint4*>(sm)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    if (c.tid < NC) {
        const uint32_t r = (uint32_t)(col0 + c.tid), j = (uint32_t)c.tid;
        *reinterpret_cast<__nv_bfloat16*>(sm + 2 * kTileB + sw128_off(r, j >> 3) + (j & 7) * 2) = __float2bfloat16_rn(1.f);
    }
    auto store = [&](int g, const uint32_t (&hi)[16], const uint32_t (&lo)[16]) {
        const size_t mi = (size_t)s * p.nseg + g;
        gstore_bf16_w16(p.sfx + ((mi * 2 + 0) * HD + c.row) * HD + col0 + c0, hi, c.row < HD);
        gstore_bf16_w16(p.sfx + ((mi * 2 + 1) * HD + c.row) * HD + col0 + c0, lo, c.row < HD);
    };
    {   // Sfx of the last range: the identity
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int x = 0; x < 16; ++x) {
            const int col = col0 + c0 + 2 * x;
            hi[x] = (col == c.row ? 0x3f80u : 0u) | (col + 1 == c.row ? 0x3f800000u : 0u);
            lo[x] = 0u;
        }
        store(p.nseg - 1, hi, lo);
    }
    fence_proxy_async_smem();
    __syncthreads();
#pragma unroll 1
    for (int g = p.nseg - 1; g >= 1 && c.ok; --g) {
        if (c.tid == 0) {
            const long mrow = ((long)s * p.nseg + g) * 2 * HD;
            mbar_expect_tx(&c.bars[0], 2 * kT * HD * 2);
            tma_tile(sm, &tm.dyh, &c.bars[0], HD, (int)mrow);
            tma_tile(sm + kTileB, &tm.dyh, &c.bars[0], HD, (int)(mrow + HD));
        }
        loads_wait(c);
        publish();
        if (c.tid == 0 && c.ok) {
            tc_fence_after_sync();
            const uint32_t a = smem_u32(sm);
            mma(c.tmem, a, OP_K, a + 2 * kTileB, OP_MN, HD / 16, NC, false);       // M R
            mma(c.tmem, a + kTileB, OP_K, a + 2 * kTileB, OP_MN, HD / 16, NC, true);
            mma(c.tmem, a, OP_K, a + 3 * kTileB, OP_MN, HD / 16, NC, true);
            umma_commit(&c.bars[1]);
        }
        mma_wait(c);
        if (!c.ok) break;
        float v[32];
        uint32_t hi[16], lo[16];
        tmem_row32(c.tl + c0, v);
        split32(v, hi, lo);
        if (c.row < HD) {
            tile_store_w16(sm + 2 * kTileB, c.row, c0, hi);
            tile_store_w16(sm + 3 * kTileB, c.row, c0, lo);
        }
        store(g - 1, hi, lo);
    }
    teardown<128>(c, p.status);
}

// ---------------------------------------------------------------------------------------------- a product applied to row tiles
// grid = S * N.  x M  for every 128-row tile of x ([S][Lp][d] bf16), with M = hi + lo from [S][nseg][2][d][d] bf16 (tm.dyh):
// the matrix of the tile's slice and, with nseg > 1, of the range of seg_chunks chunks the tile lies in.  The result
// replaces x (bf16, p.qv: the query state of the context-parallel path after a key segment has been attended, paper
// Sec. 3.5; the gate terms of the rows move on as well: gq[row] += gtot[slice]) or goes to a float32 matrix
// (p.kc, [S][cap][d]: the prompt's key cache, second pass).
template <int HD>
__global__ void __launch_bounds__(256, 2) apply_product_kernel(const __grid_constant__ LevelTensorMaps tm, const LevelParams p) {
    extern __shared__ uint8_t smem_raw[];
    Ctx c;
    setup<128>(c, smem_raw, kBar3);
    const int s = blockIdx.x / p.N, ch = blockIdx.x % p.N;
    uint8_t* sm = c.smem;   // slots: 0 x tile, 1 M hi, 2 M lo
    const long row0 = (long)s * p.Lp + (long)ch * kT;
    const long mi = p.nseg > 1 ? (long)s * p.nseg + ch / p.seg_chunks : (long)s;
    if (c.tid == 0) {
        mbar_expect_tx(&c.bars[0], 3 * kT * HD * 2);
        tma_tile(sm, &tm.qv, &c.bars[0], HD, (int)row0);
        tma_tile(sm + kTileB, &tm.dyh, &c.bars[0], HD, (int)(2 * mi * HD));
        tma_tile(sm + 2 * kTileB, &tm.dyh, &c.bars[0], HD, (int)((2 * mi + 1) * HD));
    }
    if (p.gq && c.tid < kT) p.gq[row0 + c.tid] += p.gtot[s];
    loads_wait(c);
    if (c.tid == 0 && c.ok) {
        tc_fence_after_sync();
        const uint32_t a = smem_u32(sm);
        mma(c.tmem, a, OP_K, a + kTileB, OP_MN, HD / 16, HD, false);
        mma(c.tmem, a, OP_K, a + 2 * kTileB, OP_MN, HD / 16, HD, true);
        umma_commit(&c.bars[1]);
    }
    mma_wait(c);
    if (c.ok) {
        float v[32];
        const int pos = ch * kT + c.row;
        for (int i = 0; i < HD / 64; ++i) {
            const int c0 = c.half * (HD / 2) + i * 32;
            tmem_row32(c.tl + c0, v);
            if (p.kc) gstore_f32x32(p.kc + ((size_t)s * p.cap + pos) * HD + c0, v, pos < p.L);
            else gstore_bf16x32(p.qv + ((size_t)row0 + c.row) * HD + c0, v);
        }
    }
    teardown<128>(c, p.status);
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
        case LEVEL_DYADIC_FUSED: {
            const int half_w = 1 << (p.fuse - 1);
            dim3 g(p.S * ((p.lv.dy_cnt[p.l + 1] + half_w - 1) / half_w));
            return hd == 64 ? launch(dyadic_fused_kernel<64>, g, 6, tm, p, st) : launch(dyadic_fused_kernel<128>, g, 6, tm, p, st);
        }
        case LEVEL_DYADIC_FWD: {
            dim3 g(p.S * p.lv.dy_cnt[p.l + 1]);
            return hd == 64 ? launch(dyadic_fwd_kernel<64>, g, 4, tm, p, st) : launch(dyadic_fwd_kernel<128>, g, 4, tm, p, st);
        }
        case LEVEL_VERSION_FWD: {
            dim3 g(p.S * p.N, 2);
            return hd == 64 ? launch(version_fwd_kernel<64>, g, 3, tm, p, st) : launch(version_fwd_kernel<128>, g, 3, tm, p, st);
        }
        case LEVEL_BWD: {
            dim3 g(p.S * p.lv.dy_cnt[p.l]);
            return hd == 64 ? launch(level_bwd_kernel<64>, g, 7, tm, p, st) : launch(level_bwd_kernel<128>, g, 7, tm, p, st);
        }
        case LEVEL_KEY_CACHE: {
            dim3 g(p.S, hd / 64, p.nseg > 1 ? p.nseg : 1);
            return hd == 64 ? launch(key_cache_kernel<64, false>, g, 5, tm, p, st) : launch(key_cache_kernel<128, false>, g, 5, tm, p, st);
        }
        case LEVEL_QUERY_EDGE: {
            dim3 g(p.S, hd / 64);
            return hd == 64 ? launch(key_cache_kernel<64, true>, g, 5, tm, p, st) : launch(key_cache_kernel<128, true>, g, 5, tm, p, st);
        }
        case LEVEL_SUFFIX: {
            dim3 g(p.S, hd / 64);
            return hd == 64 ? launch(suffix_kernel<64>, g, 4, tm, p, st) : launch(suffix_kernel<128>, g, 4, tm, p, st);
        }
        case LEVEL_APPLY_PRODUCT: {
            dim3 g(p.S * p.N);
            return hd == 64 ? launch(apply_product_kernel<64>, g, 3, tm, p, st) : launch(apply_product_kernel<128>, g, 3, tm, p, st);
        }
        default:
            return cudaErrorInvalidValue;
    }
}

}  // namespace path
