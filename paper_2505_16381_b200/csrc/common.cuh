// Shared declarations of the PaTH attention library's translation units.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace path {

constexpr int CHUNK = 128;  // chunk size B of the blockwise algorithm == query tile == key tile

// Codes written to the device status word when a bounded wait runs out.
enum : uint32_t {
    ST_OK = 0,
    ST_FWD_PRODUCER = 0x101, ST_FWD_MMA = 0x102, ST_FWD_SOFTMAX = 0x103,
    ST_DKV_PRODUCER = 0x201, ST_DKV_MMA = 0x202, ST_DKV_COMPUTE = 0x203,
    ST_DQ_PRODUCER = 0x301, ST_DQ_MMA = 0x302, ST_DQ_COMPUTE = 0x303,
    ST_PREP = 0x401, ST_CHAIN = 0x501, ST_LEVELS = 0x601,
    ST_GEMM = 0x801,
    ST_STATE = 0x701,      // path_attn_bwd_reuse: the workspace does not hold the forward state of this problem
    ST_SELFTEST = 0x7f1,   // path_attn_selftest_timeout: the wait it makes run out
};

// What a forward that ran on a backward-sized workspace leaves at byte kStateRecordOffset of the status block: which
// problem the chunk preparation in the workspace belongs to.  path_attn_bwd_reuse compares it on the device.
constexpr size_t kStateRecordOffset = 64;
constexpr unsigned long long kStateMagic = 0x50615448537461ull;
struct StateRecord {
    unsigned long long magic;
    const void *q, *k, *v, *w, *beta, *log_f;
    int B, H, L, d;
    float scale;   // compared for gated problems only (the block-skipping counts depend on it)
    int gate;
};

__host__ __device__ inline int msb32(unsigned x) {
#ifdef __CUDA_ARCH__
    return 31 - __clz((int)x);
#else
    int r = -1;
    while (x) { ++r; x >>= 1; }
    return r;
#endif
}
// Storage slot of the level-l version of query chunk I / key chunk J.  Slot 0 holds the
// boundary-adjusted tile itself, which is the version at the chunk's first usable level
// (lowest set bit of I, lowest clear bit of J); higher levels live in slot == level.
__host__ __device__ inline int lowest_set(unsigned x) {
#ifdef __CUDA_ARCH__
    return __ffs((int)x) - 1;
#else
    int r = 0;
    if (!x) return -1;
    while (!(x & 1u)) { ++r; x >>= 1; }
    return r;
#endif
}
__host__ __device__ inline int qslot(int level, int I) { return level == lowest_set((unsigned)I) ? 0 : level; }
__host__ __device__ inline int kslot(int level, int J) { return level == lowest_set(~(unsigned)J) ? 0 : level; }

// Where the versions live.  Plane 0 is [S][Lp][d]: every chunk's boundary-adjusted tile (= its version at its first usable
// level).  The other versions follow, packed: slice after slice, chunk after chunk, level after level.  Query chunk I
// has one per set bit of I above the lowest, key chunk J one per clear bit of J (below nlev) above the lowest, so a
// slice holds about N log2(N) / 2 extra tiles instead of N (log2(N) - 1).  All positions are closed forms of the chunk
// index (prefix sums of bit counts), so no table is stored.
__host__ __device__ inline int popcount32(unsigned x) {
#ifdef __CUDA_ARCH__
    return __popc(x);
#else
    return __builtin_popcount(x);
#endif
}
__host__ __device__ inline int popcount_prefix(unsigned n) {   // sum of popcount(c) over c = 0 .. n-1
    int total = 0;
    for (int j = 0; j < 31 && (1u << j) < n; ++j) {
        const int rem = (int)(n & ((2u << j) - 1u)) - (int)(1u << j);
        total += (int)((n >> (j + 1)) << j) + (rem > 0 ? rem : 0);
    }
    return total;
}
struct VerLayout {
    int S, N, Lp, nlev;
    int eq, ek;   // extra tiles per slice on the query / key side
};
__host__ __device__ inline int q_extra_before(int I) { return I > 0 ? popcount_prefix((unsigned)I) - (I - 1) : 0; }
__host__ __device__ inline int k_extra_before(int J, int nlev) { return nlev > 0 ? J * (nlev - 1) - popcount_prefix((unsigned)J) : 0; }
__host__ __device__ inline VerLayout make_ver_layout(int S, int N, int Lp, int nlev) {
    VerLayout v{S, N, Lp, nlev, 0, 0};
    v.eq = q_extra_before(N);
    const int last = nlev - popcount32((unsigned)(N - 1)) - 1;
    v.ek = k_extra_before(N - 1, nlev) + (last > 0 ? last : 0);
    return v;
}
// First row (in units of rows of d elements) of the level-`level` version of query chunk I / key chunk J of slice s.
__host__ __device__ inline long qver_row(const VerLayout& v, int s, int level, int I) {
    if (level == lowest_set((unsigned)I)) return (long)s * v.Lp + (long)I * CHUNK;
    const int rank = popcount32((unsigned)I & ((1u << level) - 1u)) - 1;
    return ((long)v.S * v.N + (long)s * v.eq + q_extra_before(I) + rank) * CHUNK;
}
__host__ __device__ inline long kver_row(const VerLayout& v, int s, int level, int J) {
    if (level == lowest_set(~(unsigned)J)) return (long)s * v.Lp + (long)J * CHUNK;
    const int rank = level - popcount32((unsigned)J & ((1u << level) - 1u)) - 1;
    return ((long)v.S * v.N + (long)s * v.ek + k_extra_before(J, v.nlev) + rank) * CHUNK;
}

struct FwdTensorMaps {
    CUtensorMap q_raw, k_raw, v, qv, kv, xqn, yt;  // qv/kv also serve as the low parts' maps in split mode
};

struct FwdParams {
    void* o;            // [S, L, HD] bf16 or f32
    float* lse;         // [S, L]
    const float* G;     // [S, Lp] inclusive prefix of the log gate, or nullptr
    const int* nkeep;   // [S, N] key chunks each query chunk has to visit (gated problems), or nullptr = all
    uint32_t* status;   // device status word
    int S, L, Lp, N;
    VerLayout vl;       // placement of the query / key versions behind tm.qv / tm.kv
    float scale;
    int out_fp32;
    // segment-against-segment sweep of the context-parallel path only (launch_fa_fwd_cross): the key segment's padded
    // length and chunk count, and its gate terms [S, Lkp] (G then holds the query rows' terms; logit += G_i - Gk_j)
    const float* Gk;
    int Lkp, Nk;
};

// Placement of the dyadic run products: level l holds dy_cnt[l] = N >> l matrices per slice, starting
// dy_off[l] elements into the buffer (same layout for the bf16 hi / lo planes and the float gradients).
struct LevelTable {
    long dy_off[20];
    int dy_cnt[20];
};

struct LevelTensorMaps {
    CUtensorMap dyh, dyl;   // [matrices * d][d] bf16 hi / lo planes of the run products
    CUtensorMap qv, kv;     // bf16 versions, rows of d elements placed by VerLayout
    CUtensorMap dqv, dkv;   // same shape: bf16 gradients of the versions (backward only)
    CUtensorMap ddy;        // [matrices * d][d] bf16 gradients of the run products (backward only)
};

struct LevelParams {
    LevelTable lv;
    VerLayout vl;
    int l;                  // dyadic forward: level consumed (l -> l + 1); version forward: number of levels; level backward: the
                            // level of the run products whose gradients the launch finishes
    int nlev;               // number of levels (level backward)
    int fuse;               // fused dyadic forward: levels l + 1 .. l + fuse are produced by one launch (2 or 3)
    int S, N, Lp;
    __nv_bfloat16 *dyh, *dyl, *qv, *kv;
    __nv_bfloat16 *dqv, *dkv;     // gradients of the versions (placed like them); plane 0 ends up holding the final sums
    __nv_bfloat16* ddy16;         // gradients of the run products, same placement as the run products themselves
    float* kc;                    // edge kernels: [S][cap][d] float32 out (rows < L of every slice), or nullptr
    int cap, L;
    __nv_bfloat16* edge16;        // edge kernels: [S][L][d] bf16 out, or nullptr
    __nv_bfloat16* pseg;          // edge kernels: [S][nseg][2][d][d] product of the walked range as bf16 hi, lo; or nullptr
    __nv_bfloat16* sfx;           // suffix kernel: [S][nseg][2][d][d] out
    int nseg, seg_chunks;         // key-side edge / suffix / apply-product kernels: ranges per slice (<= 1: none), chunks per range
    float* gq;                    // apply-product kernel: [S][Lp] gate terms of the rows (+= gtot[slice]), or nullptr
    const float* gtot;            // [S]
    const int *nkeep, *nvisit;    // version backward: chunk counts of a sweep shortened by block skipping ([S][N]), or nullptr
    uint32_t* status;
};

enum { LEVEL_DYADIC_FWD = 0, LEVEL_DYADIC_FUSED, LEVEL_VERSION_FWD, LEVEL_BWD, LEVEL_KEY_CACHE, LEVEL_QUERY_EDGE, LEVEL_SUFFIX, LEVEL_APPLY_PRODUCT };
cudaError_t launch_level_kernel(int which, const LevelTensorMaps& tm, const LevelParams& p, int hd, cudaStream_t st);

struct PrepTensorMaps {
    CUtensorMap w, q, k;   // [S*Lp][d] bf16, box 128 rows x 64 columns, 128-byte swizzle
    // stores of the tiles kept for the chain rule (backward's instance only): [S*Lp][128]; u is [S*Lp][d]
    CUtensorMap th, tl, xk, u;
};

struct PrepParams {
    const float* beta;            // [S*Lp] (zero in the ragged tail)
    const __nv_bfloat16* q;       // [S*Lp][d]
    const __nv_bfloat16* k;
    __nv_bfloat16* ql;            // [S*Lp][d]   boundary-adjusted queries (version slot 0)
    __nv_bfloat16* kr;            // [S*Lp][d]   boundary-adjusted keys (version slot 0)
    __nv_bfloat16* Xqn;           // [S*Lp][128] -lower(Q W^T)
    __nv_bfloat16* Yt;            // [S*Lp][128] (T~ strictLower(W K^T))^T
    __nv_bfloat16 *Ph, *Pl;       // [S*N][d][d] chunk products as a bf16 hi + lo pair (level 0 of the run products)
    // (I + N)^-1 as a bf16 hi + lo pair for the chain rule, written only by the backward's instance ([S*Lp][128]);
    // that instance also keeps T~ (hi + lo) and Xk, U rounded once, through the tensor maps
    __nv_bfloat16 *sAh, *sAl;
    uint32_t* status;
};

// `mode`: what the kernel produces (see chunk_prep.cu).
enum { PREP_FWD = 0, PREP_SAVE = 1, PREP_KEYS = 2 };
cudaError_t launch_chunk_prep(const PrepTensorMaps& tm, const PrepParams& p, int hd, int mode, int nchunks,
                              cudaStream_t st);

struct ChainTensorMaps {
    CUtensorMap w, q, k, u;                       // [S*Lp][d]
    CUtensorMap yt, xqn, xk, th, tl, ah, al;      // [S*Lp][128]; yt = Y^T and xqn = -Xq are the attention sweep's operands
    CUtensorMap dsdt;                             // [S*N*128][128] bf16: (scale * lower(dS))^T of the diagonal chunks
    CUtensorMap dql, dkr;                         // [S*Lp][d] bf16 gradients of the boundary-adjusted queries / keys
    CUtensorMap dp;                               // [S*N*d][d] bf16 gradients of the chunk products
};

struct ChainParams {
    const __nv_bfloat16* dql;   // [S*Lp][d]  gradient of the boundary-adjusted queries (version slot 0), bf16
    const __nv_bfloat16* dkr;   // [S*Lp][d]  gradient of the boundary-adjusted keys, bf16
    const float* beta;    // [S*Lp]
    __nv_bfloat16 *dq, *dk, *dw;   // [S][L][d] outputs
    float* dbeta;         // [S][L]
    uint32_t* status;
    int N, L;
    float scale;
};

cudaError_t launch_chunk_chain(const ChainTensorMaps& tm, const ChainParams& p, int hd, int nchunks, cudaStream_t st);

struct BwdTensorMaps {
    CUtensorMap q_raw, k_raw, v, qv, kv, xqn, yt, d_o;
};

struct BwdParams {
    VerLayout vl;        // placement of the versions and of their gradients
    __nv_bfloat16* dqv;  // gradients of the query versions (placed like the versions), bf16
    __nv_bfloat16* dkv;  // same for the key versions
    void* dv;            // [S, L, d] bf16, final
    float* dsd;          // [S*N][128 q][128 k] lower(dS) of the diagonal chunks, unscaled; written for gated problems only
    __nv_bfloat16* dsdt; // [S*N][128 k][128 q] (scale * lower(dS))^T in bf16: the chain rule's operand
    float* dG;           // [S][Lp] minus the column sums of dS (gated problems only)
    float* dGrow;        // [S][Lp] row sums of dS over the off-diagonal chunks (gated problems only)
    const float* lse2;   // [S][Lp] (gate prefix - lse) * log2(e)
    const float* delta;  // [S][Lp] -(dO . O)
    const float* G;      // [S][Lp] gate prefix or nullptr
    const int* nkeep;    // [S][N] key chunks a query chunk has to visit / nvisit: query chunks a key chunk has to meet
    const int* nvisit;   //        (block skipping in gated problems), or nullptr = all
    uint32_t* status;
    int S, L, Lp, N;
    float scale;
};

cudaError_t launch_fa_bwd(const BwdTensorMaps& tm, const BwdParams& p, int hd, int which, cudaStream_t st);
cudaError_t launch_rowstats(const void* o, const void* d_o, const float* lse, const float* G, float* delta, float* lse2,
                            int S, int L, int Lp, int hd, cudaStream_t st);
cudaError_t launch_fa_fwd(const FwdTensorMaps& tm, const FwdParams& p, int hd, cudaStream_t st);
// Every query chunk of one segment against every key chunk of another (tm.qv / tm.kv / tm.v only; p.G, p.Gk required).
cudaError_t launch_fa_fwd_cross(const FwdTensorMaps& tm, const FwdParams& p, int hd, cudaStream_t st);
// One decoding step over an in-place float32 key cache (paper Sec. 3.4); `part` holds decode_partials_bytes(S, cap, hd).
size_t decode_partials_bytes(int S, int cap, int hd);
cudaError_t launch_decode_step(const void* q_t, const void* k_t, const void* v_t, const void* w_t, const float* beta_t,
                               const float* log_f_t, float* kc, void* vc, float* gc, int t, int cap, void* o_t, float* lse_t,
                               int S, int hd, float scale, float* part, cudaStream_t st);
// Float32 forward by the definition (PATH_FP32): q, k, v, w, o are [S][L][hd] float, G the gate prefix [S][ldG] or nullptr.
cudaError_t launch_fp32_fwd(const float* q, const float* k, const float* v, const float* w, const float* beta, const float* G,
                            float* o, float* lse, int S, int L, int ldG, int hd, float scale, cudaStream_t st);
// Layer front-end (paper Sec. 2.2 footnote, Sec. 2.4 gate): z [B][L][H*hd] bf16 and logits [B][L][H] -> w [B][H][L][hd] bf16,
// beta / log f [B][H][L]; and the backward (dcw must be zero on entry: CTAs add into it).
cudaError_t launch_frontend_fwd(const void* z, const float* cw, const float* bl, const float* gl, void* w, float* beta,
                                float* logf, int B, int H, int L, int hd, float eps, cudaStream_t st);
cudaError_t launch_frontend_bwd(const void* z, const float* cw, const float* bl, const float* gl, const void* dw,
                                const float* dbeta, const float* dlogf, void* dz, float* dcw, float* dbl, float* dgl, int B,
                                int H, int L, int hd, float eps, cudaStream_t st);

// One product C[M, N] (+)= op(A) op(B) of the low-rank layer (lowrank.cu).  a_mn / b_mn: the operand is stored as
// [K][rows] (tensor map box 64 x 64) instead of [rows][K] (box 128 rows x 64).  c: bf16 [M][ldc] overwritten, or, with
// c_atomic, float32 [M][ldc] added to.
struct GemmParams {
    int M, N, K;
    int a_mn, b_mn;
    void* c;
    int ldc, c_atomic;
    uint32_t* status;
};
cudaError_t launch_gemm(const CUtensorMap& map_a, const CUtensorMap& map_b, const GemmParams& p, int split_k, cudaStream_t st);

}  // namespace path
