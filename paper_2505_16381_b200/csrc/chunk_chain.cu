// Per-chunk chain rule of the backward pass (the paper gives no backward): from the gradients of the
// boundary-adjusted tiles (dQl, dKr), of the diagonal-chunk logits (dSd) and of the chunk product (dP) back through
// the UT transform to dq, dk, dw, dbeta.  With Xq = lower(Q W^T), Xk = strictLower(W K^T), Y = T~ Xk, U = T~ W,
// T~ = Ainv D, Ainv = (I + strictLower(D W W^T))^-1 and s = scale:
//   dXq = lower(-dQl U^T - s dSd Y^T)            dY  = -W dKr^T - s Xq^T dSd           dU = -Xq^T dQl - W dP
//   dT  = lower(dY Xk^T + dU W^T)                dXk = strictLower(T~^T dY)
//   M   = Ainv^T dT,   dbeta_c  = M_cc,          dA  = strictLower(-(M D) Ainv^T)
//   dbeta_r += sum_c dA_rc (W W^T)_rc,           dGm = D dA
//   dq = dQl + s dSd K + dXq W                   dk = dKr + s dSd^T Q + dXk^T W
//   dw = -Y dKr - U dP^T + T~^T dU + dXq^T Q + dXk K + (dGm + dGm^T) W
// A persistent CTA (one per SM) walks over chunks and runs these ~31 products per chunk as tcgen05 MMAs on swizzled
// shared-memory tiles.  Eight worker warps turn accumulators (tensor memory, one row per thread) into the next operand
// tiles; the first lane of a ninth warp requests every tile (TMA) and issues every product.  The two sides meet only
// through mbarriers: the workers hand tiles over and go on (they wait for products, never for the issuer), the issuer
// sends out first whatever does not depend on the read-out in progress, starts the next chunk's first products while
// the current chunk's results are still leaving, and requests tiles the moment their slots are free.  dQl and dKr
// arrive as bf16 tiles.  T~ and Ainv enter as bf16 hi + lo pairs, and so do the in-kernel intermediates dT, M D and dGm;
// everything else is rounded to bf16 once.  dw accumulates in tensor memory across all phases.
#include "tileops.cuh"

namespace path {
using namespace tile;

namespace {

constexpr int kSlots = 7;
constexpr int kChainThreads = 288;   // eight worker warps + the warp whose first lane loads tiles and issues products
constexpr uint32_t kBarOff = kSlots * kTileB;
constexpr uint32_t kChainSmem = kBarOff + 64 + kT * 4 + kT * 4 + 1024;

template <int HD>
__global__ void __launch_bounds__(kChainThreads, 1) chunk_chain_kernel(const __grid_constant__ ChainTensorMaps tm,
                                                             const ChainParams p, const int nchunks) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(smem + kBarOff);  // two for loads, two for product groups, two for the workers' hand-overs
    uint32_t* tmem_slot = (uint32_t*)(bars + 6);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float* bt = (float*)(smem + kBarOff + 64);
    float* t1 = bt + kT;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row = (warp & 3) * 32 + lane, half = (warp >> 2) & 1;

    if (tid == 0) {
        for (int i = 0; i < 6; ++i) mbar_init(&bars[i], i < 4 ? 1u : 256u);   // B_R0, B_R1: every worker arrives
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(tmem_slot, 512);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    auto slot = [&](int i) { return smem + i * kTileB; };
    auto sa = [&](int i) { return smem_u32(smem + i * kTileB); };
    constexpr int KD = HD / 16, K8 = 8;
    constexpr uint32_t cDW = 0, cA = 128, cB = 256, cG = 384;   // tensor-memory columns: dw, two work accumulators, W W^T
    enum { B_LOAD = 0, B_LOAD2, B_MMA, B_MMA2, B_R0, B_R1, B_COUNT };
    const int grid = (int)gridDim.x;

    if (warp == 8) {
    if (lane == 0) {
    // ------------------------------------------------------------------ leader: TMA loads and every product
    bool ok = true;
    uint32_t ph[7] = {0, 0, 0, 0, 0, 0, 0};
    auto wait = [&](int b) {   // false (and nothing more is issued) once a wait has run out
        if (ok && !mbar_wait(&bars[b], ph[b], abort_flag, ST_CHAIN)) ok = false;
        ph[b] ^= 1;
        tc_fence_after_sync();
        return ok;
    };
    // slots: 0 U->dXq   1 dQl->T~ hi->Ainv hi->K   2 Y^T->-Xq->Xk->dT hi->tmp hi->dGm hi   3 dSd->T~ lo->dT lo->tmp lo->dSd
    //        4 W   5 dKr->dY->dXk->dGm lo   6 dP->dU->Ainv lo->Q
    // First tiles of a chunk, in two parts: five of the seven slots are free as soon as the products that finish dq and dk
    // have retired, and these five tiles are all that the chunk's first two products read; the other two slots feed the
    // previous chunk's very last products.
    auto first_loads_a = [&](int ch) {
        mbar_expect_tx(&bars[B_LOAD], 3 * kT * HD * 2 + 2 * kTileB);
        tma_tile(slot(1), &tm.dql, &bars[B_LOAD], HD, ch * kT);
        tma_tile(slot(0), &tm.u, &bars[B_LOAD], HD, ch * kT);
        tma_tile(slot(3), &tm.dsdt, &bars[B_LOAD], kT, ch * kT);   // (s dSd)^T: every use takes the transposed view
        tma_tile(slot(2), &tm.yt, &bars[B_LOAD], kT, ch * kT);
        tma_tile(slot(6), &tm.dp, &bars[B_LOAD], HD, ch * HD);
    };
    auto first_loads_b = [&](int ch) {
        mbar_expect_tx(&bars[B_LOAD2], 2 * kT * HD * 2);
        tma_tile(slot(5), &tm.dkr, &bars[B_LOAD2], HD, ch * kT);
        tma_tile(slot(4), &tm.w, &bars[B_LOAD2], HD, ch * kT);
    };
    if ((int)blockIdx.x < nchunks) {
        first_loads_a(blockIdx.x);
        first_loads_b(blockIdx.x);
    }
#pragma unroll 1
    for (int chunk = blockIdx.x; chunk < nchunks && ok; chunk += grid) {
        const int r0 = chunk * kT;
        // ---- phase 0: dXq = lower(-(dQl U^T + s dSd Y^T)) -> cA, while the previous chunk's results are still leaving
        // the other columns; then dw = -Y dKr - U dP^T
        if (!wait(B_LOAD)) break;
        mma_call(tmem + cA, sa(1), OP_K, sa(0), OP_K, KD, 128, false);
        mma_call(tmem + cA, sa(3), OP_MN, sa(2), OP_MN, K8, 128, true);          // slot 2 holds Y^T
        if (chunk != (int)blockIdx.x && !wait(B_R1)) break;                      // the previous chunk's dw has left cDW
        if (!wait(B_LOAD2)) break;
        mma_call(tmem + cDW, sa(2), OP_MN, sa(5), OP_MN, K8, HD, false, true);
        mma_call(tmem + cDW, sa(0), OP_K, sa(6), OP_K, KD, HD, true, true);
        umma_commit(&bars[B_MMA]);
        // ---- phase 1: dY = -(W dKr^T + Xq^T s dSd) -> cA,  dU = -(Xq^T dQl + W dP) -> cB.  dU's products read no tile
        // that the workers are writing and go to their own columns: they run underneath the read-out of dXq.
        if (!wait(B_MMA)) break;
        mbar_expect_tx(&bars[B_LOAD], kTileB);
        tma_tile(slot(2), &tm.xqn, &bars[B_LOAD], kT, r0);
        mma_call(tmem + cB, sa(4), OP_K, sa(6), OP_MN, KD, HD, false);           // W dP needs no new tile
        if (!wait(B_LOAD)) break;
        mma_call(tmem + cB, sa(2), OP_MN, sa(1), OP_MN, K8, HD, true, true);     // slot 2 holds -Xq: negated back
        if (!wait(B_R0)) break;                                                  // dXq has left cA
        mma_call(tmem + cA, sa(4), OP_K, sa(5), OP_K, KD, 128, false);
        mma_call(tmem + cA, sa(2), OP_MN, sa(3), OP_K, K8, 128, true, true);
        umma_commit(&bars[B_MMA]);
        // ---- phase 2: dT = lower(dY Xk^T + dU W^T) -> cA, and phase 3 right behind it (the same dY and dU tiles and T~):
        // dXk = strictLower(T~^T dY) -> cB,  dw += T~^T dU.  (s dSd)^T is not needed again before phase 5, where it is
        // loaded once more: until then its slot (3) takes the lo parts of the bf16 pairs.
        if (!wait(B_MMA)) break;
        mbar_expect_tx(&bars[B_LOAD], 3 * kTileB);
        tma_tile(slot(2), &tm.xk, &bars[B_LOAD], kT, r0);
        tma_tile(slot(1), &tm.th, &bars[B_LOAD], kT, r0);
        tma_tile(slot(3), &tm.tl, &bars[B_LOAD], kT, r0);
        if (!wait(B_R1)) break;                                                  // dY, dU tiles
        mma_call(tmem + cA, sa(6), OP_K, sa(4), OP_K, KD, 128, false);           // dU W^T needs no new tile
        if (!wait(B_LOAD)) break;
        mma_call(tmem + cA, sa(5), OP_K, sa(2), OP_K, K8, 128, true);
        umma_commit(&bars[B_MMA]);
        mma_call(tmem + cB, sa(1), OP_MN, sa(5), OP_MN, K8, 128, false);
        mma_call(tmem + cB, sa(3), OP_MN, sa(5), OP_MN, K8, 128, true);
        mma_call(tmem + cDW, sa(1), OP_MN, sa(6), OP_MN, K8, HD, true);
        mma_call(tmem + cDW, sa(3), OP_MN, sa(6), OP_MN, K8, HD, true);
        umma_commit(&bars[B_MMA2]);
        // ---- phase 4: M = Ainv^T dT -> cG;  tmp = M D;  dA = strictLower(-tmp Ainv^T) -> cA;  W W^T -> cB (for dbeta)
        if (!wait(B_MMA) || !wait(B_MMA2)) break;
        mbar_expect_tx(&bars[B_LOAD], 2 * kTileB);
        tma_tile(slot(1), &tm.ah, &bars[B_LOAD], kT, r0);
        tma_tile(slot(6), &tm.al, &bars[B_LOAD], kT, r0);
        if (!wait(B_LOAD)) break;
        if (!wait(B_R0)) break;                                                  // dT hi, lo tiles
        mma_call(tmem + cG, sa(1), OP_MN, sa(2), OP_MN, K8, 128, false);
        mma_call(tmem + cG, sa(6), OP_MN, sa(2), OP_MN, K8, 128, true);
        mma_call(tmem + cG, sa(1), OP_MN, sa(3), OP_MN, K8, 128, true);
        umma_commit(&bars[B_MMA]);
        if (!wait(B_R1)) break;                                                  // dXk has left cB
        mma_call(tmem + cB, sa(4), OP_K, sa(4), OP_K, KD, 128, false);          // retires with the next group
        if (!wait(B_MMA)) break;
        if (!wait(B_R0)) break;                                                  // tmp hi, lo tiles
        mma_call(tmem + cA, sa(2), OP_K, sa(1), OP_K, K8, 128, false);
        mma_call(tmem + cA, sa(2), OP_K, sa(6), OP_K, K8, 128, true);
        mma_call(tmem + cA, sa(3), OP_K, sa(1), OP_K, K8, 128, true);
        umma_commit(&bars[B_MMA]);
        // ---- phase 5: dq -> cB, dk -> cG and the rest of dw, in three groups.  K and Q replace Ainv hi / lo, (s dSd)^T
        // returns.  First the products that need neither dGm nor the columns that dbeta still reads; when they have
        // retired, dXk's slot is free for dGm lo.  The second group finishes dq and dk, the third (dGm lo) only dw.
        if (!wait(B_MMA)) break;
        mbar_expect_tx(&bars[B_LOAD], 2 * kT * HD * 2 + kTileB);
        tma_tile(slot(3), &tm.dsdt, &bars[B_LOAD], kT, r0);
        tma_tile(slot(6), &tm.q, &bars[B_LOAD], HD, r0);
        tma_tile(slot(1), &tm.k, &bars[B_LOAD], HD, r0);
        mma_call(tmem + cG, sa(5), OP_MN, sa(4), OP_MN, K8, HD, false);          // dXk^T W needs no new tile
        if (!wait(B_LOAD)) break;
        mma_call(tmem + cG, sa(3), OP_K, sa(6), OP_MN, K8, HD, true);            // s dSd^T Q
        mma_call(tmem + cDW, sa(0), OP_MN, sa(6), OP_MN, K8, HD, true);          // dXq^T Q
        mma_call(tmem + cDW, sa(5), OP_K, sa(1), OP_MN, K8, HD, true);           // dXk K
        umma_commit(&bars[B_MMA2]);
        if (!wait(B_R1)) break;                                                  // dGm hi tile; W W^T has left cB
        mma_call(tmem + cB, sa(3), OP_MN, sa(1), OP_MN, K8, HD, false);          // s dSd K
        mma_call(tmem + cB, sa(0), OP_K, sa(4), OP_MN, K8, HD, true);            // dXq W
        mma_call(tmem + cDW, sa(2), OP_K, sa(4), OP_MN, K8, HD, true);           // dGm W
        mma_call(tmem + cDW, sa(2), OP_MN, sa(4), OP_MN, K8, HD, true);          // dGm^T W
        umma_commit(&bars[B_MMA]);
        if (!wait(B_MMA2)) break;
        // (the last two products cannot start before the second group has left the pipe anyway: the next chunk's tiles are
        // requested first, the moment their slots are free)
        const int next = chunk + grid;
        if (!wait(B_MMA)) break;
        if (next < nchunks) first_loads_a(next);                                 // slots 0 - 3 and 6 are free
        if (!wait(B_R0)) break;                                                  // dGm lo tile (over dXk)
        mma_call(tmem + cDW, sa(5), OP_K, sa(4), OP_MN, K8, HD, true);
        mma_call(tmem + cDW, sa(5), OP_MN, sa(4), OP_MN, K8, HD, true);
        umma_commit(&bars[B_MMA2]);
        if (!wait(B_MMA2)) break;
        if (next < nchunks) first_loads_b(next);                                 // and the other two
    }
    }
    __syncwarp();
    } else {
    // ------------------------------------------------------------------ workers: accumulators -> next operand tiles
    bool ok = true;
    uint32_t ph_mma = 0, ph_mma2 = 0;
    float v[32];
    auto wsync_and = [&](bool good) {   // barrier over the eight worker warps + AND of `good`
        uint32_t r;
        __syncwarp();
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.b32 p, %1, 0;\n\t"
            "bar.red.and.pred q, 1, 256, p;\n\t"
            "selp.u32 %0, 1, 0, q;\n\t}"
            : "=r"(r)
            : "r"((uint32_t)good)
            : "memory");
        return r != 0;
    };
    auto wsync = [&]() {
        __syncwarp();
        asm volatile("bar.sync 1, 256;" ::: "memory");
    };
    // lane 0 of every warp waits for the product group; the vote that follows releases the other lanes
    auto mma_wait = [&](int b = B_MMA) {
        uint32_t& ph = b == B_MMA ? ph_mma : ph_mma2;
        bool good = true;
        if (lane == 0) good = mbar_wait(&bars[b], ph, abort_flag, ST_CHAIN);
        ph ^= 1;
        ok = wsync_and(good);
        tc_fence_after_sync();
    };
    // tiles written by this thread become visible to the MMA unit, its accumulator reads are ordered, the leader learns
    auto publish = [&](int b) {
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&bars[b]);
    };
    // accumulator [128][ncols] -> f(row values) -> bf16 tile
    enum { M_NONE = 0, M_LOWER = 1, M_STRICT = 2 };
    auto acc_to_tile = [&](uint32_t col, int ncols, uint8_t* dst, float mul, int mask) {
        const int per = ncols / 2;
        for (int c = 0; c < per / 32; ++c) {
            const int c0 = half * per + c * 32;
            tmem_row32(tl + col + c0, v);
#pragma unroll
            for (int x = 0; x < 32; ++x) {
                const bool keep = mask == M_NONE || (mask == M_LOWER ? (c0 + x <= row) : (c0 + x < row));
                v[x] = keep ? v[x] * mul : 0.f;
            }
            tile_store32(dst, row, c0, v);
        }
    };
    // accumulator [128][128] -> f(value, column) -> hi or lo part of its bf16 pair -> tile
    auto split_to_tile = [&](uint32_t col, uint8_t* dst, bool want_lo, auto&& f) {
        for (int c = 0; c < 2; ++c) {
            const int c0 = half * 64 + c * 32;
            tmem_row32(tl + col + c0, v);
#pragma unroll
            for (int x = 0; x < 32; ++x) {
                const float t = f(v[x], c0 + x);
                const float h = __bfloat162float(__float2bfloat16_rn(t));
                v[x] = want_lo ? t - h : h;
            }
            tile_store32(dst, row, c0, v);
        }
    };
    // the same, both parts from one read of the accumulator
    auto split_both = [&](uint32_t col, uint8_t* dst_hi, uint8_t* dst_lo, auto&& f) {
        for (int c = 0; c < 2; ++c) {
            const int c0 = half * 64 + c * 32;
            uint32_t hi[16], lo[16];
            tmem_row32(tl + col + c0, v);
#pragma unroll
            for (int x = 0; x < 32; ++x) v[x] = f(v[x], c0 + x);
            split32(v, hi, lo);
            tile_store_w16(dst_hi, row, c0, hi);
            tile_store_w16(dst_lo, row, c0, lo);
        }
    };
    auto f_dT = [&](float x, int col) { return col <= row ? x : 0.f; };
    auto f_tmp = [&](float x, int col) { return x * bt[col]; };
    auto f_dGm = [&](float x, int col) { return col < row ? -bt[row] * x : 0.f; };

#pragma unroll 1
    for (int chunk = blockIdx.x; chunk < nchunks; chunk += grid) {
        const int s_idx = chunk / p.N, pos = (chunk % p.N) * kT + row;   // slice and position of this thread's row
        const bool row_valid = pos < p.L;
        const size_t urow = (size_t)s_idx * p.L + pos;                   // row in the caller's [S][L][.] tensors
        if (tid < kT) bt[tid] = p.beta[(size_t)chunk * kT + tid];   // first read after several barriers (phase 4)
        mma_wait();                                                 // phase 0
        if (!ok) break;
        acc_to_tile(cA, kT, slot(0), -1.f, M_LOWER);                // dXq (over U)
        publish(B_R0);
        mma_wait();                                                 // phase 1
        if (!ok) break;
        acc_to_tile(cA, kT, slot(5), -1.f, M_NONE);                 // dY (over dKr)
        acc_to_tile(cB, HD, slot(6), -1.f, M_NONE);                 // dU (over dP)
        publish(B_R1);
        mma_wait();                                                 // phase 2
        if (!ok) break;
        // dT stays in tensor memory (cA); its bf16 hi part goes over Xk now, the lo part follows once T~ lo has been read
        split_to_tile(cA, slot(2), false, f_dT);
        mma_wait(B_MMA2);                                           // phase 3
        if (!ok) break;
        split_to_tile(cA, slot(3), true, f_dT);                     // dT lo (over T~ lo)
        publish(B_R0);
        // dXk leaves its columns while M is being computed; W W^T takes them over as soon as it has
        acc_to_tile(cB, kT, slot(5), 1.f, M_STRICT);                // dXk (over dY)
        publish(B_R1);
        mma_wait();                                                 // M
        if (!ok) break;
        {   // diagonal of M -> t1 (dbeta's column part)
            const int c0 = (row >> 5) << 5;
            if ((c0 >> 6) == half) {
                tmem_row32(tl + cG + c0, v);
#pragma unroll
                for (int x = 0; x < 32; ++x)
                    if (c0 + x == row) t1[row] = v[x];
            }
        }
        split_both(cG, slot(2), slot(3), f_tmp);                    // tmp = M D, hi (over dT hi) and lo (over dT lo)
        publish(B_R0);
        mma_wait();                                                 // dA and W W^T
        if (!ok) break;
        float dbeta_row;
        {   // dA = strictLower(-cA);  dbeta_r = t1_r + sum_c dA_rc (W W^T)_rc
            float part = 0.f;
            for (int c = 0; c < 2; ++c) {
                const int c0 = half * 64 + c * 32;
                float gm[32];
                tmem_row32(tl + cA + c0, v);
                tmem_row32(tl + cB + c0, gm);
#pragma unroll
                for (int x = 0; x < 32; ++x)
                    if (c0 + x < row) part -= v[x] * gm[x];
            }
            // the two threads of a row add their halves through shared memory
            wsync();
            if (half == 1) t1[row] += part;
            wsync();
            dbeta_row = t1[row] + part;
        }
        split_to_tile(cA, slot(2), false, f_dGm);                   // dGm = D dA, hi
        publish(B_R1);
        // (global stores and loads come after a hand-over, never just before it: the hand-over waits for them)
        if (half == 0 && row_valid) p.dbeta[urow] = dbeta_row;
        // The dQl / dKr rows of the final sums are fetched while the products run.  At d = 128 a thread's half row is one
        // 128-byte line: four lanes fetch four lines together, a quarter of each per instruction (whole lines per request
        // instead of 32 scattered pieces, which held up the products' operand reads as well).
        constexpr int NI = HD / 64;
        uint32_t rq[4][8], rk[4][8];
        uint4 pre_q[4], pre_k[4];
        {
            const __nv_bfloat16* g_dql = p.dql + ((size_t)chunk * kT + row) * HD + half * (HD / 2);
            const __nv_bfloat16* g_dkr = p.dkr + ((size_t)chunk * kT + row) * HD + half * (HD / 2);
            if (HD == 128) {
                gload_f32x32_issue(reinterpret_cast<const float*>(g_dql), rq);
                gload_f32x32_issue(reinterpret_cast<const float*>(g_dkr), rk);
            } else {
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    pre_q[x] = reinterpret_cast<const uint4*>(g_dql)[x];
                    pre_k[x] = reinterpret_cast<const uint4*>(g_dkr)[x];
                }
            }
        }
        mma_wait(B_MMA2);                                           // phase 5, first group: dXk's slot is free
        if (!ok) break;
        split_to_tile(cA, slot(5), true, f_dGm);                    // dGm lo (over dXk)
        publish(B_R0);
        mma_wait();                                                 // phase 5, second group
        if (!ok) break;
        // dq and dk are complete: they leave while the last two products run
        {
            float wq[32], wk[32];   // HD == 128: the fetched half rows, two bf16 per word
            if (HD == 128) {
                gload_f32x32_finish(rq, wq);
                gload_f32x32_finish(rk, wk);
            }
            auto add_row = [&](const float (&words)[32], const uint4 (&pre)[4], int c, float (&acc)[32]) {
                if (HD == 128) {
#pragma unroll
                    for (int x = 0; x < 16; ++x) {
                        const uint32_t u = __float_as_uint(words[16 * c + x]);
                        acc[2 * x] += __uint_as_float(u << 16);
                        acc[2 * x + 1] += __uint_as_float(u & 0xffff0000u);
                    }
                } else {
                    float in[32];
                    unpack_bf16x32(pre, in);
#pragma unroll
                    for (int x = 0; x < 32; ++x) acc[x] += in[x];
                }
            };
#pragma unroll
            for (int c = 0; c < NI; ++c) {
                const int c0 = half * (HD / 2) + c * 32;
                tmem_row32(tl + cB + c0, v);
                add_row(wq, pre_q, c, v);
                gstore_bf16x32(p.dq + urow * HD + c0, v, row_valid);
                tmem_row32(tl + cG + c0, v);
                add_row(wk, pre_k, c, v);
                gstore_bf16x32(p.dk + urow * HD + c0, v, row_valid);
            }
        }
        mma_wait(B_MMA2);                                           // the last of dw
        if (!ok) break;
#pragma unroll
        for (int c = 0; c < NI; ++c) {
            const int c0 = half * (HD / 2) + c * 32;
            tmem_row32(tl + cDW + c0, v);
            gstore_bf16x32(p.dw + urow * HD + c0, v, row_valid);
        }
        publish(B_R1);   // the next chunk's first products overwrite the accumulators read above
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

cudaError_t launch_chunk_chain(const ChainTensorMaps& tm, const ChainParams& p, int hd, int nchunks, cudaStream_t st) {
    int dev = 0, sms = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    e0 = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e0 != cudaSuccess) return e0;
    const int grid = nchunks < sms ? nchunks : sms;
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kChainSmem);
        if (e != cudaSuccess) return e;
        kern<<<grid, kChainThreads, kChainSmem, st>>>(tm, p, nchunks);
        return cudaGetLastError();
    };
    return hd == 64 ? go(chunk_chain_kernel<64>) : go(chunk_chain_kernel<128>);
}

}  // namespace path
