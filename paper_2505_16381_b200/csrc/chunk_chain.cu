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
// A persistent CTA (one per SM) walks over chunks and runs these ~25 products per chunk as tcgen05 MMAs on swizzled
// shared-memory tiles, in lockstep: thread 0 loads tiles (TMA) and issues MMAs, all 256 threads turn accumulators
// (tensor memory, one row per thread) into the next operand tiles.  dQl and dKr arrive as bf16 tiles; the next
// chunk's first tiles are requested before the current chunk's results are written out.  T~ and Ainv enter as bf16
// hi + lo pairs, and so do the in-kernel intermediates dT, M D and dGm (the lo tile follows the hi tile through
// the same slot); everything else is rounded to bf16 once.  dw accumulates in tensor memory across all phases.
#include "tileops.cuh"

namespace path {
using namespace tile;

namespace {

constexpr int kSlots = 7;
constexpr uint32_t kBarOff = kSlots * kTileB;
constexpr uint32_t kChainSmem = kBarOff + 64 + kT * 4 + kT * 4 + 1024;

template <int HD>
__global__ void __launch_bounds__(256, 1) chunk_chain_kernel(const __grid_constant__ ChainTensorMaps tm,
                                                             const ChainParams p, const int nchunks) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(smem + kBarOff);  // [0] loads, [1] MMA groups
    uint32_t* tmem_slot = (uint32_t*)(bars + 2);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    float* bt = (float*)(smem + kBarOff + 64);
    float* t1 = bt + kT;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row = (warp & 3) * 32 + lane, half = warp >> 2;

    if (tid == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
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
    bool ok = true;
    uint32_t ph_load = 0, ph_mma = 0;
    float v[32];

    // thread 0: start TMA loads of bf16 tiles; everyone: wait for them
    auto loads_wait = [&]() {
        if (!mbar_wait(&bars[0], ph_load, abort_flag, ST_CHAIN)) ok = false;
        ph_load ^= 1;
    };
    // everyone: tiles written by threads become visible to the MMA unit, accumulator reads are ordered
    auto publish = [&]() {
        fence_proxy_async_smem();
        tc_fence_before_sync();
        __syncthreads();
    };
    auto mma_wait = [&]() {
        __syncwarp();
        if (!mbar_wait(&bars[1], ph_mma, abort_flag, ST_CHAIN)) ok = false;
        ph_mma ^= 1;
        ok = __syncthreads_and(ok);
        tc_fence_after_sync();
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

    // slots: 0 U->W   1 dQl->dT->tmp->dGm   2 Y^T->-Xq->Xk->T->Ah->K   3 dSd->T lo->dT lo->tmp lo->dSd   4 dXq   5 dKr->dY->dXk
    //        6 dP->dU->Al->Q
    // first tiles of a chunk: U, Y, (s dSd)^T (every use below takes the transposed view), dQl, dKr, dP
    // They are requested in two parts: four of the six slots are free as soon as phase 5's products have retired, the
    // other two (0, 1) feed the chunk's very last products.  All bytes are announced with the first part.
    auto first_loads_a = [&](int ch) {
        mbar_expect_tx(&bars[0], 4 * kT * HD * 2 + 2 * kTileB);
        tma_tile(slot(6), &tm.dp, &bars[0], HD, ch * HD);
        tma_tile(slot(2), &tm.yt, &bars[0], kT, ch * kT);
        tma_tile(slot(3), &tm.dsdt, &bars[0], kT, ch * kT);
        tma_tile(slot(5), &tm.dkr, &bars[0], HD, ch * kT);
    };
    auto first_loads_b = [&](int ch) {
        tma_tile(slot(0), &tm.u, &bars[0], HD, ch * kT);
        tma_tile(slot(1), &tm.dql, &bars[0], HD, ch * kT);
    };
    if (tid == 0 && (int)blockIdx.x < nchunks) {
        first_loads_a(blockIdx.x);
        first_loads_b(blockIdx.x);
    }
#pragma unroll 1
    for (int chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
    const int s_idx = chunk / p.N, pos = (chunk % p.N) * kT + row;   // slice and position of this thread's row
    const bool row_valid = pos < p.L;
    const size_t urow = (size_t)s_idx * p.L + pos;                   // row in the caller's [S][L][.] tensors
    const __nv_bfloat16* g_dql = p.dql + ((size_t)chunk * kT + row) * HD;
    const __nv_bfloat16* g_dkr = p.dkr + ((size_t)chunk * kT + row) * HD;
    const int r0 = chunk * kT;
    if (tid < kT) bt[tid] = p.beta[(size_t)chunk * kT + tid];   // first read after several barriers (phase 4)
    // ---- phase 0a: dXq = lower(-(dQl U^T + s dSd Y^T))
    loads_wait();
    publish();
    if (tid == 0) {
        tc_fence_after_sync();
        mma_call(tmem + cA, sa(1), OP_K, sa(0), OP_K, KD, 128, false);
        mma_call(tmem + cA, sa(3), OP_MN, sa(2), OP_MN, K8, 128, true);          // slot 2 holds Y^T
        // phase 0b: dw = -Y dKr - U dP^T
        mma_call(tmem + cDW, sa(2), OP_MN, sa(5), OP_MN, K8, HD, false, true);
        mma_call(tmem + cDW, sa(0), OP_K, sa(6), OP_K, KD, HD, true, true);
        umma_commit(&bars[1]);
    }
    mma_wait();
    if (!ok) break;
    // ---- phase 1: dY = -(W dKr^T + Xq^T s dSd),  dU = -(Xq^T dQl + W dP),  Gm = W W^T
    // (every group's tiles are requested as soon as the products that read the slots have retired, before the
    // read-out of the accumulators, so that the TMA latency hides behind it)
    if (tid == 0) {
        mbar_expect_tx(&bars[0], kT * HD * 2 + kTileB);
        tma_tile(slot(0), &tm.w, &bars[0], HD, r0);
        tma_tile(slot(2), &tm.xqn, &bars[0], kT, r0);
    }
    acc_to_tile(cA, kT, slot(4), -1.f, M_LOWER);                    // dXq
    loads_wait();
    publish();
    if (tid == 0) {
        tc_fence_after_sync();
        mma_call(tmem + cA, sa(0), OP_K, sa(5), OP_K, KD, 128, false);
        mma_call(tmem + cA, sa(2), OP_MN, sa(3), OP_K, K8, 128, true, true);     // slot 2 holds -Xq: negated back
        mma_call(tmem + cB, sa(2), OP_MN, sa(1), OP_MN, K8, HD, false, true);
        mma_call(tmem + cB, sa(0), OP_K, sa(6), OP_MN, KD, HD, true);
        mma_call(tmem + cG, sa(0), OP_K, sa(0), OP_K, KD, 128, false);
        umma_commit(&bars[1]);
    }
    mma_wait();
    if (!ok) break;
    // ---- phase 2: dT = lower(dY Xk^T + dU W^T)
    if (tid == 0) {
        mbar_expect_tx(&bars[0], kTileB);
        tma_tile(slot(2), &tm.xk, &bars[0], kT, r0);
    }
    acc_to_tile(cA, kT, slot(5), -1.f, M_NONE);                     // dY (over dKr)
    acc_to_tile(cB, HD, slot(6), -1.f, M_NONE);                     // dU (over dP)
    loads_wait();
    publish();
    if (tid == 0) {
        tc_fence_after_sync();
        mma_call(tmem + cA, sa(5), OP_K, sa(2), OP_K, K8, 128, false);
        mma_call(tmem + cA, sa(6), OP_K, sa(0), OP_K, KD, 128, true);
        umma_commit(&bars[1]);
    }
    mma_wait();
    if (!ok) break;
    // ---- phase 3: dXk = strictLower(T~^T dY) -> cB,  dw += T~^T dU.  (s dSd)^T is not needed again before phase 5, where
    // it is loaded once more: until then its slot (3) takes the lo parts of the bf16 pairs, so that the hi and lo products
    // of a pair go out as one group.
    if (tid == 0) {
        mbar_expect_tx(&bars[0], 2 * kTileB);
        tma_tile(slot(2), &tm.th, &bars[0], kT, r0);
        tma_tile(slot(3), &tm.tl, &bars[0], kT, r0);
    }
    // dT stays in tensor memory (cA); its bf16 hi part goes to slot 1 now, the lo part follows in phase 4
    split_to_tile(cA, slot(1), false, f_dT);
    loads_wait();
    publish();
    if (tid == 0) {
        tc_fence_after_sync();
        mma_call(tmem + cB, sa(2), OP_MN, sa(5), OP_MN, K8, 128, false);
        mma_call(tmem + cB, sa(3), OP_MN, sa(5), OP_MN, K8, 128, true);
        mma_call(tmem + cDW, sa(2), OP_MN, sa(6), OP_MN, K8, HD, true);
        mma_call(tmem + cDW, sa(3), OP_MN, sa(6), OP_MN, K8, HD, true);
        umma_commit(&bars[1]);
    }
    mma_wait();
    if (!ok) break;
    // ---- phase 4: M = Ainv^T dT -> cB;  dbeta_c = M_cc;  tmp = M D;  dA = strictLower(-tmp Ainv^T) -> cA
    if (tid == 0) {
        mbar_expect_tx(&bars[0], 2 * kTileB);
        tma_tile(slot(2), &tm.ah, &bars[0], kT, r0);
        tma_tile(slot(6), &tm.al, &bars[0], kT, r0);
    }
    acc_to_tile(cB, kT, slot(5), 1.f, M_STRICT);                    // dXk (over dY)
    split_to_tile(cA, slot(3), true, f_dT);                         // dT lo (over T~ lo)
    loads_wait();
    publish();
    if (tid == 0) {
        tc_fence_after_sync();
        mma_call(tmem + cB, sa(2), OP_MN, sa(1), OP_MN, K8, 128, false);
        mma_call(tmem + cB, sa(6), OP_MN, sa(1), OP_MN, K8, 128, true);
        mma_call(tmem + cB, sa(2), OP_MN, sa(3), OP_MN, K8, 128, true);
        umma_commit(&bars[1]);
    }
    mma_wait();
    if (!ok) break;
    {   // diagonal of M -> t1
        const int c0 = (row >> 5) << 5;
        if ((c0 >> 6) == half) {
            tmem_row32(tl + cB + c0, v);
#pragma unroll
            for (int x = 0; x < 32; ++x)
                if (c0 + x == row) t1[row] = v[x];
        }
    }
    split_both(cB, slot(1), slot(3), f_tmp);                        // tmp = M D, hi (over dT hi) and lo (over dT lo)
    publish();
    if (tid == 0) {
        tc_fence_after_sync();
        mma_call(tmem + cA, sa(1), OP_K, sa(2), OP_K, K8, 128, false);
        mma_call(tmem + cA, sa(1), OP_K, sa(6), OP_K, K8, 128, true);
        mma_call(tmem + cA, sa(3), OP_K, sa(2), OP_K, K8, 128, true);
        umma_commit(&bars[1]);
    }
    mma_wait();
    if (!ok) break;
    if (tid == 0) {   // phase 5's K and Q replace Ainv hi / lo, whose last products have just retired; (s dSd)^T returns
        mbar_expect_tx(&bars[0], 2 * kT * HD * 2 + kTileB);
        tma_tile(slot(2), &tm.k, &bars[0], HD, r0);
        tma_tile(slot(6), &tm.q, &bars[0], HD, r0);
        tma_tile(slot(3), &tm.dsdt, &bars[0], kT, r0);
    }
    {   // dA = strictLower(-cA);  dbeta_r = t1_r + sum_c dA_rc Gm_rc
        float part = 0.f;
        for (int c = 0; c < 2; ++c) {
            const int c0 = half * 64 + c * 32;
            float gm[32];
            tmem_row32(tl + cA + c0, v);
            tmem_row32(tl + cG + c0, gm);
#pragma unroll
            for (int x = 0; x < 32; ++x)
                if (c0 + x < row) part -= v[x] * gm[x];
        }
        // the two threads of a row add their halves through shared memory
        __syncthreads();
        if (half == 1) t1[row] += part;
        __syncthreads();
        if (half == 0 && row_valid) p.dbeta[urow] = t1[row] + part;
    }
    split_to_tile(cA, slot(1), false, f_dGm);                       // dGm = D dA, hi
    // ---- phase 5: dq -> cB, dk -> cG and the rest of dw
    loads_wait();
    publish();
    if (tid == 0) {
        tc_fence_after_sync();
        mma_call(tmem + cB, sa(3), OP_MN, sa(2), OP_MN, K8, HD, false);   // s dSd K
        mma_call(tmem + cB, sa(4), OP_K, sa(0), OP_MN, K8, HD, true);     // dXq W
        mma_call(tmem + cG, sa(3), OP_K, sa(6), OP_MN, K8, HD, false);    // s dSd^T Q
        mma_call(tmem + cG, sa(5), OP_MN, sa(0), OP_MN, K8, HD, true);    // dXk^T W
        mma_call(tmem + cDW, sa(4), OP_MN, sa(6), OP_MN, K8, HD, true);   // dXq^T Q
        mma_call(tmem + cDW, sa(5), OP_K, sa(2), OP_MN, K8, HD, true);    // dXk K
        mma_call(tmem + cDW, sa(1), OP_K, sa(0), OP_MN, K8, HD, true);    // dGm W
        mma_call(tmem + cDW, sa(1), OP_MN, sa(0), OP_MN, K8, HD, true);   // dGm^T W
        umma_commit(&bars[1]);
    }
    mma_wait();
    if (!ok) break;
    if (tid == 0 && chunk + (int)gridDim.x < nchunks) first_loads_a(chunk + gridDim.x);   // slots 2, 3, 5, 6 are free
    split_to_tile(cA, slot(1), true, f_dGm);                        // dGm lo
    publish();
    if (tid == 0) {
        tc_fence_after_sync();
        mma_call(tmem + cDW, sa(1), OP_K, sa(0), OP_MN, K8, HD, true);
        mma_call(tmem + cDW, sa(1), OP_MN, sa(0), OP_MN, K8, HD, true);
        umma_commit(&bars[1]);
    }
    // the dQl / dKr rows of the final sums are fetched while the last products run
    constexpr int NI = HD / 64;
    uint4 pre_q[NI][4], pre_k[NI][4];
#pragma unroll
    for (int c = 0; c < NI; ++c) {
        const int c0 = half * (HD / 2) + c * 32;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            pre_q[c][x] = reinterpret_cast<const uint4*>(g_dql + c0)[x];
            pre_k[c][x] = reinterpret_cast<const uint4*>(g_dkr + c0)[x];
        }
    }
    mma_wait();
    if (!ok) break;
    // every product of this chunk has retired: the last two slots are free for the next chunk's first tiles
    if (tid == 0 && chunk + (int)gridDim.x < nchunks) first_loads_b(chunk + gridDim.x);
#pragma unroll
    for (int c = 0; c < NI; ++c) {
        const int c0 = half * (HD / 2) + c * 32;
        float in[32];
        tmem_row32(tl + cB + c0, v);
        unpack_bf16x32(pre_q[c], in);
#pragma unroll
        for (int x = 0; x < 32; ++x) v[x] += in[x];
        gstore_bf16x32(p.dq + urow * HD + c0, v, row_valid);
        tmem_row32(tl + cG + c0, v);
        unpack_bf16x32(pre_k[c], in);
#pragma unroll
        for (int x = 0; x < 32; ++x) v[x] += in[x];
        gstore_bf16x32(p.dk + urow * HD + c0, v, row_valid);
        tmem_row32(tl + cDW + c0, v);
        gstore_bf16x32(p.dw + urow * HD + c0, v, row_valid);
    }
    // the next chunk's first products overwrite the accumulators read above
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    }   // chunk loop

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
        kern<<<grid, 256, kChainSmem, st>>>(tm, p, nchunks);
        return cudaGetLastError();
    };
    return hd == 64 ? go(chunk_chain_kernel<64>) : go(chunk_chain_kernel<128>);
}

}  // namespace path
