// The low-rank linear layer in front of the short convolution (paper Sec. 2.2, footnote to the definition of H_t: w_t
// comes from "a low-rank linear layer followed by a short convolution and L2 normalisation"):
//     t = x W1^T   [M, r],      z = t W2^T   [M, C]        (x [M, D];  W1 [r, D],  W2 [C, r]:  nn.Linear layouts)
// and its backward
//     dt = dz W2,   dW2 = dz^T t,   dx = dt W1,   dW1 = dt^T x.
// All six are one tcgen05 kernel: C[M', N'] (+)= op(A) op(B) on 128 x 128 output tiles, operands fetched by TMA into a
// three-stage ring of 128-byte-swizzled tiles, one thread issuing the products into a tensor-memory accumulator, four
// warps writing the tile out.  Whether an operand enters as stored or transposed is a matter of its descriptor's
// major-ness, as everywhere in this library: a K-major operand is a [rows][K] matrix (box 128 rows x 64 k), an MN-major
// one a [K][rows] matrix (box 64 k x 64 rows, two per stage).  The weight gradients contract over the M tokens: their
// K range is split over CTAs and the partial tiles are added with float32 atomics (reproducible to rounding).
// These products have a short contraction or a narrow output: they are bound by the bytes of x, z and their
// gradients, not by the tensor pipe.
#include "tileops.cuh"

namespace path {
using namespace tc5;

namespace {

constexpr int kStages = 3;   // 3 x 32 KB: two CTAs per SM, so one writes its tile out while the other multiplies
constexpr uint32_t kStageBytes = 32768;   // A tile [128 x 64] + B tile [128 x 64], bf16
constexpr uint32_t kGemmSmem = kStages * kStageBytes + 256 + 1024;

// Descriptor low words of the k-th 16-wide step inside a 64-deep stage tile.
__device__ __forceinline__ uint32_t step_lo(uint32_t tile, int mn_major, int kk) {
    // K-major: [128 rows][64 k], 32 bytes per step.  MN-major: two panels [64 k][64 rows], 8192 bytes apart, 2048 bytes per step.
    return mn_major ? umma_desc_lo(tile + kk * 2048u, 8192u) : umma_desc_lo(tile + kk * 32u, 16u);
}

__global__ void __launch_bounds__(192, 2) gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                                                      const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full = (uint64_t*)(smem + kStages * kStageBytes);
    uint64_t* empty = full + kStages;
    uint64_t* done = empty + kStages;
    uint32_t* tmem_slot = (uint32_t*)(done + 1);
    volatile uint32_t* abort_flag = (volatile uint32_t*)(tmem_slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
        mbar_init(done, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(tmem_slot, 128);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    const int m0 = blockIdx.x * 128, n0 = blockIdx.y * 128;
    // this CTA's share of the contraction, in stages of 64
    const int stages_total = (p.K + 63) / 64, per = (stages_total + (int)gridDim.z - 1) / (int)gridDim.z;
    const int s_lo = blockIdx.z * per, s_hi = min(stages_total, s_lo + per), ns = s_hi - s_lo;
    if (warp == 0 && lane == 0) {
        // ---------------------------------------------------------------- producer
        bool ok = true;
        for (int i = 0; i < ns && ok; ++i) {
            const int st = i % kStages, k0 = (s_lo + i) * 64;
            if (i >= kStages && !mbar_wait(&empty[st], ((i / kStages) - 1) & 1, abort_flag, ST_GEMM)) { ok = false; break; }
            uint8_t* a = smem + st * kStageBytes;
            uint8_t* b = a + 16384;
            mbar_expect_tx(&full[st], kStageBytes);
            if (p.a_mn) { tma_load_2d(a, &map_a, &full[st], m0, k0); tma_load_2d(a + 8192, &map_a, &full[st], m0 + 64, k0); }
            else tma_load_2d(a, &map_a, &full[st], k0, m0);
            if (p.b_mn) { tma_load_2d(b, &map_b, &full[st], n0, k0); tma_load_2d(b + 8192, &map_b, &full[st], n0 + 64, k0); }
            else tma_load_2d(b, &map_b, &full[st], k0, n0);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------------------------------------------------------- product issue
        const uint32_t idesc = umma_idesc(128, 128, p.a_mn, p.b_mn);
        bool ok = true;
        for (int i = 0; i < ns && ok; ++i) {
            const int st = i % kStages;
            if (!mbar_wait(&full[st], (i / kStages) & 1, abort_flag, ST_GEMM)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t a = smem_u32(smem + st * kStageBytes), b = a + 16384;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                umma_ss(tmem, umma_desc_join(step_lo(a, p.a_mn, kk)), umma_desc_join(step_lo(b, p.b_mn, kk)), idesc,
                        (i > 0 || kk > 0) ? 1u : 0u);
            umma_commit(&empty[st]);
        }
        if (ok) umma_commit(done);
    } else if (warp >= 2) {
        // ---------------------------------------------------------------- write-out: one row per thread
        const int q4 = warp & 3, row = q4 * 32 + lane, m = m0 + row;
        const uint32_t tl = tmem + ((uint32_t)(q4 * 32) << 16);
        bool ok = ns > 0 ? mbar_wait(done, 0, abort_flag, ST_GEMM) : true;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after_sync();
        if (ok) {
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                const int n = n0 + c * 32;
                if (n >= p.N) break;
                float v[32];
                if (ns > 0) tile::tmem_row32(tl + c * 32, v);
                else {
#pragma unroll
                    for (int x = 0; x < 32; ++x) v[x] = 0.f;
                }
                if (p.c_atomic) {
                    if (m < p.M && ns > 0) {
                        float* dst = (float*)p.c + (size_t)m * p.ldc + n;
#pragma unroll
                        for (int x = 0; x < 32; ++x)
                            if (n + x < p.N) atomicAdd(dst + x, v[x]);
                    }
                } else {   // bf16, N a multiple of 32 (checked on the host)
                    tile::gstore_bf16x32((__nv_bfloat16*)p.c + (size_t)(m < p.M ? m : 0) * p.ldc + n, v, m < p.M);
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && *abort_flag != 0) atomicCAS(p.status, 0u, *abort_flag);
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem, 128);
    }
}

}  // namespace

cudaError_t launch_gemm(const CUtensorMap& map_a, const CUtensorMap& map_b, const GemmParams& p, int split_k, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGemmSmem);
    if (e != cudaSuccess) return e;
    dim3 grid((p.M + 127) / 128, (p.N + 127) / 128, split_k);
    gemm_kernel<<<grid, 192, kGemmSmem, st>>>(map_a, map_b, p);
    return cudaGetLastError();
}

}  // namespace path
