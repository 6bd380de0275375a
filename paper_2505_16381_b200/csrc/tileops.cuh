// Building blocks of the per-chunk kernels: every matrix of the chunk-level algebra is a 128-row
// bf16 tile in shared memory (row-major, 64-column panels, 128-byte swizzle), every product a tcgen05 MMA into
// tensor memory issued by one thread, every result read back one row per thread (256 worker threads: two per row,
// each taking half of the columns).
#pragma once
#include "common.cuh"
#include "tc5.cuh"

namespace path {
namespace tile {
using namespace tc5;

constexpr int kT = 128;
constexpr uint32_t kTileB = 32768, kPanelB = 16384;

// K view: contraction over the tile's columns.  MN view: contraction over the tile's rows.
enum { OP_K = 0, OP_MN = 1 };
__device__ __forceinline__ uint64_t desc_k(uint32_t t, int kk) {
    return umma_desc(t + (kk >> 2) * kPanelB + (kk & 3) * 32, 16, 1024);
}
__device__ __forceinline__ uint64_t desc_mn(uint32_t t, int kk) { return umma_desc(t + kk * 2048, kPanelB, 1024); }

// D[128 x n] (+)= (+-) op(A) op(B), `ksteps` steps of 16 along the contraction.  One thread issues all of them, so the
// instructions between two tcgen05.mma count: only the low word of a descriptor changes from step to step (the start
// address; the strides and the swizzle mode sit in the high word), by a constant the view decides.
__device__ __forceinline__ void mma(uint32_t d_tmem, uint32_t a_tile, int a_op, uint32_t b_tile, int b_op, int ksteps,
                                    int n, bool acc, bool negate = false) {
    const uint32_t idesc = umma_idesc(128, n, a_op, b_op) | (negate ? (1u << 13) : 0u);
    uint32_t a_lo = umma_desc_lo(a_tile, a_op == OP_K ? 16u : kPanelB);
    uint32_t b_lo = umma_desc_lo(b_tile, b_op == OP_K ? 16u : kPanelB);
    // K view: 32 bytes per step, the next 64-column panel after four; MN view: 2048 bytes per step
    const uint32_t a_step = a_op == OP_K ? 2u : 128u, a_jump = a_op == OP_K ? (kPanelB - 96u) >> 4 : 128u;
    const uint32_t b_step = b_op == OP_K ? 2u : 128u, b_jump = b_op == OP_K ? (kPanelB - 96u) >> 4 : 128u;
    uint32_t accum = acc ? 1u : 0u;
    for (int kk = 0; kk < ksteps; ++kk) {
        umma_ss(d_tmem, umma_desc_join(a_lo), umma_desc_join(b_lo), idesc, accum);
        accum = 1u;
        const bool last_of_panel = (kk & 3) == 3;
        a_lo += last_of_panel ? a_jump : a_step;
        b_lo += last_of_panel ? b_jump : b_step;
    }
}

// The products of a kernel whose issuing thread lives on a small register allotment (setmaxnreg): descriptors rebuilt at
// every step, nothing carried across the loop.
__device__ __forceinline__ void mma_small(uint32_t d_tmem, uint32_t a_tile, int a_op, uint32_t b_tile, int b_op, int ksteps,
                                          int n, bool acc, bool negate = false) {
    const uint32_t idesc = umma_idesc(128, n, a_op, b_op) | (negate ? (1u << 13) : 0u);
    for (int kk = 0; kk < ksteps; ++kk)
        umma_ss(d_tmem, a_op == OP_K ? desc_k(a_tile, kk) : desc_mn(a_tile, kk),
                b_op == OP_K ? desc_k(b_tile, kk) : desc_mn(b_tile, kk), idesc, (acc || kk > 0) ? 1u : 0u);
}

// The same as a real function, for kernels that issue dozens of different products from straight-line code: inlined,
// they no longer fit the instruction cache (and the issuing thread's small register allotment).
static __device__ __noinline__ void mma_call(uint32_t d_tmem, uint32_t a_tile, int a_op, uint32_t b_tile, int b_op, int ksteps,
                                             int n, bool acc, bool negate = false) {
    mma(d_tmem, a_tile, a_op, b_tile, b_op, ksteps, n, acc, negate);
}

// Stores columns c0 .. c0+31 of `row` of a swizzled bf16 tile.
__device__ __forceinline__ void tile_store32(uint8_t* t, int row, int c0, const float (&v)[32]) {
    uint8_t* panel = t + (c0 >> 6) * kPanelB;
    const int ch0 = (c0 & 63) >> 3;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch)
        *reinterpret_cast<uint4*>(panel + sw128_off((uint32_t)row, (uint32_t)(ch0 + ch))) =
            make_uint4(pack_bf16(v[8 * ch], v[8 * ch + 1]), pack_bf16(v[8 * ch + 2], v[8 * ch + 3]),
                       pack_bf16(v[8 * ch + 4], v[8 * ch + 5]), pack_bf16(v[8 * ch + 6], v[8 * ch + 7]));
}
// Row transfers between registers and global memory.  Lane L of a warp owns one row segment (32 consecutive values
// starting at its own pointer).  All 32 lanes must call together: the lanes of a group first swap 32-byte pieces so
// that one instruction covers whole rows (full 128- or 64-byte runs) instead of 32 scattered 16-byte pieces.
// `valid` = false: the lane's row is not written / reads as zero.
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t (&v)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]),
                 "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
__device__ __forceinline__ void ld_global_v8(const void* p, uint32_t (&v)[8]) {
    asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "l"(p)
                 : "memory");
}
__device__ __forceinline__ void gstore_f32x32(float* dst, const float (&v)[32], bool valid = true) {
    const int j = threadIdx.x & 3;
    uint32_t w[32];
#pragma unroll
    for (int x = 0; x < 32; ++x) w[x] = __float_as_uint(v[x]);
    rot4_pieces(w, j);
    const unsigned long long mine = (unsigned long long)dst;
#pragma unroll
    for (int r = 0; r < 4; ++r) {   // piece j of the row of lane (L ^ r)
        uint32_t d[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) d[x] = r == 0 ? w[x] : __shfl_xor_sync(0xffffffffu, w[8 * r + x], r);
        const unsigned long long ptr = r == 0 ? mine : __shfl_xor_sync(0xffffffffu, mine, r);
        const bool ok = r == 0 ? valid : (bool)__shfl_xor_sync(0xffffffffu, (int)valid, r);
        if (ok) st_global_v8((uint8_t*)ptr + 32 * j, d);
    }
}
// The load in two halves, so that a caller can put other work between the request and the first use of the data.
__device__ __forceinline__ void gload_f32x32_issue(const float* src, uint32_t (&d)[4][8], bool valid = true) {
    const int j = threadIdx.x & 3;
    const unsigned long long mine = (unsigned long long)src;
    unsigned long long ptr[4];
    bool ok[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        ptr[r] = r == 0 ? mine : __shfl_xor_sync(0xffffffffu, mine, r);
        ok[r] = r == 0 ? valid : (bool)__shfl_xor_sync(0xffffffffu, (int)valid, r);
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {   // all four loads are in flight together
#pragma unroll
        for (int x = 0; x < 8; ++x) d[r][x] = 0u;
        if (ok[r]) ld_global_v8((const uint8_t*)ptr[r] + 32 * j, d[r]);
    }
}
__device__ __forceinline__ void gload_f32x32_finish(const uint32_t (&d)[4][8], float (&v)[32]) {
    const int j = threadIdx.x & 3;
    uint32_t w[32];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int x = 0; x < 8; ++x) w[8 * r + x] = r == 0 ? d[r][x] : __shfl_xor_sync(0xffffffffu, d[r][x], r);
    rot4_pieces(w, j);
#pragma unroll
    for (int x = 0; x < 32; ++x) v[x] = __uint_as_float(w[x]);
}
__device__ __forceinline__ void gload_f32x32(const float* src, float (&v)[32], bool valid = true) {
    uint32_t d[4][8];
    gload_f32x32_issue(src, d, valid);
    gload_f32x32_finish(d, v);
}
// 32 bf16 = 64 bytes per row: pairs of lanes.  `w`: the row segment as 16 packed words.
__device__ __forceinline__ void gstore_bf16_w16(__nv_bfloat16* dst, const uint32_t (&w)[16], bool valid = true) {
    const bool odd = threadIdx.x & 1;
    uint32_t first[8], second[8];   // halves [32 * odd, +32) of the even lane's row and of the odd lane's row
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        const uint32_t recv = __shfl_xor_sync(0xffffffffu, odd ? w[x] : w[8 + x], 1);
        first[x] = odd ? recv : w[x];
        second[x] = odd ? w[8 + x] : recv;
    }
    const unsigned long long mine = (unsigned long long)dst, other = __shfl_xor_sync(0xffffffffu, mine, 1);
    const bool ovalid = (bool)__shfl_xor_sync(0xffffffffu, (int)valid, 1);
    if (odd ? ovalid : valid) st_global_v8((uint8_t*)(odd ? other : mine) + 32 * (int)odd, first);
    if (odd ? valid : ovalid) st_global_v8((uint8_t*)(odd ? mine : other) + 32 * (int)odd, second);
}
__device__ __forceinline__ void pack32(const float (&v)[32], uint32_t (&w)[16]) {
#pragma unroll
    for (int x = 0; x < 16; ++x) w[x] = pack_bf16(v[2 * x], v[2 * x + 1]);
}
__device__ __forceinline__ void gstore_bf16x32(__nv_bfloat16* dst, const float (&v)[32], bool valid = true) {
    uint32_t w[16];
    pack32(v, w);
    gstore_bf16_w16(dst, w, valid);
}
// t = hi + lo with hi = bf16(t) and lo = bf16(t - hi), both packed two per word.
__device__ __forceinline__ void split32(const float (&t)[32], uint32_t (&hi)[16], uint32_t (&lo)[16]) {
#pragma unroll
    for (int x = 0; x < 16; ++x) {
        const uint32_t h = pack_bf16(t[2 * x], t[2 * x + 1]);
        hi[x] = h;
        lo[x] = pack_bf16(t[2 * x] - __uint_as_float(h << 16), t[2 * x + 1] - __uint_as_float(h & 0xffff0000u));
    }
}
// Packed counterpart of tile_store32.
__device__ __forceinline__ void tile_store_w16(uint8_t* t, int row, int c0, const uint32_t (&w)[16]) {
    uint8_t* panel = t + (c0 >> 6) * kPanelB;
    const int ch0 = (c0 & 63) >> 3;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch)
        *reinterpret_cast<uint4*>(panel + sw128_off((uint32_t)row, (uint32_t)(ch0 + ch))) =
            make_uint4(w[4 * ch], w[4 * ch + 1], w[4 * ch + 2], w[4 * ch + 3]);
}
__device__ __forceinline__ void unpack_bf16x32(const uint4 (&u4)[4], float (&v)[32]) {
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const uint32_t w[4] = {u4[x].x, u4[x].y, u4[x].z, u4[x].w};
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[y]));
            v[8 * x + 2 * y] = f.x;
            v[8 * x + 2 * y + 1] = f.y;
        }
    }
}
__device__ __forceinline__ void tmem_row32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    tmem_ld32(taddr, r);
    tmem_ld_wait();
#pragma unroll
    for (int x = 0; x < 32; ++x) v[x] = __uint_as_float(r[x]);
}
// TMA load of a [128 x ncols] bf16 tile (ncols = 64 or 128) whose first row is `row0` of the mapped matrix.
__device__ __forceinline__ void tma_tile(uint8_t* dst, const CUtensorMap* m, uint64_t* bar, int ncols, int row0) {
    for (int h = 0; h < ncols / 64; ++h) tma_load_2d(dst + h * kPanelB, m, bar, h * 64, row0);
}

}  // namespace tile
}  // namespace path
