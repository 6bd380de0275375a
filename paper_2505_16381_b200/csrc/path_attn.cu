// C-ABI entry points of the PaTH attention library: argument validation, workspace planning, tensor-map
// encoding and the launch sequence.  All arithmetic runs in the kernels of linear.cu / fa_fwd.cu / fa_bwd.cu.
#include "../../include/path_attn.h"

#include <cstdio>
#include <cstring>

#include "common.cuh"
#include "linear.cuh"

namespace path {

static thread_local int g_last_cuda_error = 0;
static thread_local int g_launches = 0;

#define CK(expr)                                                  \
    do {                                                          \
        cudaError_t e__ = (expr);                                 \
        if (e__ != cudaSuccess) {                                 \
            g_last_cuda_error = (int)e__;                         \
            return PATH_ERR_LAUNCH;                               \
        }                                                         \
    } while (0)
#define LAUNCH(expr) do { CK(expr); ++g_launches; } while (0)

// ------------------------------------------------------------------------------------------- stage timing
// Optional per-thread instrumentation: CUDA events around groups of launches of the most recent call.
enum Stage { STG_PREP = 0, STG_FA_FWD, STG_PREP_BWD, STG_ROWSTATS, STG_FA_DKV, STG_FA_DQ, STG_CHAINS, STG_COUNT };
static const char* const kStageNames[STG_COUNT] = {"chunk_prep", "fa_fwd", "bwd_chunk_prep", "rowstats", "fa_bwd_dkv",
                                                   "fa_bwd_dq", "bwd_chains"};
struct Profiler {
    bool on = false, created = false;
    cudaEvent_t ev[2 * STG_COUNT];
    bool used[STG_COUNT];
};
static thread_local Profiler g_prof;

static void prof_reset(int first = 0, int last = STG_COUNT) {
    for (int i = first; i < last; ++i) g_prof.used[i] = false;
}
static void prof_mark(int stage, int end, cudaStream_t st) {
    if (!g_prof.on) return;
    if (!g_prof.created) {
        for (int i = 0; i < 2 * STG_COUNT; ++i) cudaEventCreate(&g_prof.ev[i]);
        g_prof.created = true;
    }
    cudaEventRecord(g_prof.ev[2 * stage + end], st);
    if (end) g_prof.used[stage] = true;
}

// ------------------------------------------------------------------------------------------- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 matrix [rows][cols] (row pitch = cols), box = [128 rows][64 cols], 128-byte swizzle.
static bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ------------------------------------------------------------------------------------------- workspace plan
struct Plan {
    int S, L, Lp, N, d, nlev, nslot, gate, bwd, ragged;
    LevelTable lv;
    size_t total;
    // offsets (bytes)
    size_t status, qp, kp, vp, wp, betap, G, Gm, Ai, Tt, U, Dy, Xq, Xk, Y, Xqn, Yt, Qv16, Kv16;
    // backward only
    size_t dop, delta, lse2, dQv, dKv, dSd, dG, dGrow, dGdiag, dDy, dXq, dY, dT, dXk, tmpBB, dA, dU, tq, tk, tw, t1;
    size_t dy_bytes;
};

static size_t bump(size_t& cur, size_t bytes) {
    size_t o = cur;
    cur += (bytes + 255) & ~(size_t)255;
    return o;
}

static bool make_plan(int B, int H, int L, int d, int dt, int gate, int bwd, Plan& p) {
    if (B < 1 || H < 1 || L < 1 || (d != 64 && d != 128)) return false;
    if (dt != PATH_BF16 && dt != PATH_FP32) return false;
    const long long S = (long long)B * H;
    const long long Lp = ((long long)L + CHUNK - 1) / CHUNK * CHUNK;
    if (S > (1 << 20) || Lp > (1 << 22) || S * Lp > (1LL << 31) / 16) return false;
    memset(&p, 0, sizeof(p));
    p.S = (int)S; p.L = L; p.Lp = (int)Lp; p.N = (int)(Lp / CHUNK); p.d = d; p.gate = gate; p.bwd = bwd;
    p.nlev = p.N > 1 ? msb32((unsigned)(p.N - 1)) + 1 : 0;
    p.nslot = p.nlev > 0 ? p.nlev : 1;
    p.ragged = (L != p.Lp);
    size_t cur = 0;
    const size_t SLd = (size_t)S * Lp * d, SL = (size_t)S * Lp, SNBB = (size_t)S * p.N * CHUNK * CHUNK;
    p.status = bump(cur, 256);
    if (p.ragged) {
        p.qp = bump(cur, SLd * 2); p.kp = bump(cur, SLd * 2); p.vp = bump(cur, SLd * 2); p.wp = bump(cur, SLd * 2);
    }
    p.betap = bump(cur, SL * 4);
    if (gate) p.G = bump(cur, SL * 4);
    const size_t keep = bwd ? 1 : 0;   // float intermediates of the chunk preparation, kept for the chain rule
    p.Gm = bump(cur, keep * SNBB * 4);
    p.Ai = bump(cur, keep * SNBB * 4);
    p.Tt = bump(cur, keep * SNBB * 4);
    p.U = bump(cur, keep * SLd * 4);
    size_t dy_elems = 0;
    for (int l = 0; l < 20; ++l) {
        p.lv.dy_off[l] = (long)dy_elems;
        p.lv.dy_cnt[l] = p.N >> l;
        if (l == 0 || l <= p.nlev - 2) dy_elems += (size_t)S * (p.N >> l) * d * d;
    }
    p.Dy = bump(cur, dy_elems * 4);
    p.Xq = bump(cur, keep * SNBB * 4);
    p.Xk = bump(cur, keep * SNBB * 4);
    p.Y = bump(cur, keep * SNBB * 4);
    p.Xqn = bump(cur, SL * CHUNK * 2);
    p.Yt = bump(cur, SL * CHUNK * 2);
    p.Qv16 = bump(cur, SLd * 2 * p.nslot);
    p.Kv16 = bump(cur, SLd * 2 * p.nslot);
    p.dy_bytes = dy_elems * 4;
    if (bwd) {
        if (p.ragged) p.dop = bump(cur, SLd * 2);
        p.delta = bump(cur, SL * 4); p.lse2 = bump(cur, SL * 4);
        p.dQv = bump(cur, SLd * 4 * p.nslot); p.dKv = bump(cur, SLd * 4 * p.nslot);
        p.dSd = bump(cur, SNBB * 4); p.dG = bump(cur, SL * 4);
        p.dGrow = bump(cur, gate ? SL * 4 : 0); p.dGdiag = bump(cur, gate ? SL * 4 : 0);
        p.dDy = bump(cur, dy_elems * 4);
        p.dXq = bump(cur, SNBB * 4); p.dY = bump(cur, SNBB * 4); p.dT = bump(cur, SNBB * 4);
        p.dXk = bump(cur, SNBB * 4); p.tmpBB = bump(cur, SNBB * 4); p.dA = bump(cur, SNBB * 4);
        p.dU = bump(cur, SLd * 4); p.tq = bump(cur, SLd * 4); p.tk = bump(cur, SLd * 4); p.tw = bump(cur, SLd * 4);
        p.t1 = bump(cur, SL * 4);
    }
    p.total = cur;
    return true;
}

template <class T>
static T* at(void* ws, size_t off) { return reinterpret_cast<T*>((char*)ws + off); }

static AffineBatch chunk_batch(const Plan& p, long a, long b, long c, long c2, long dd) {
    // one batch entry per chunk, buffers padded: single stride per pointer
    AffineBatch ab{};
    ab.nb1 = 1 << 30;  // z0 = 0, z1 = z
    ab.a1 = a; ab.b1 = b; ab.c1 = c; ab.c21 = c2; ab.d1 = dd;
    return ab;
}

// Chunk preparation + dyadic run products + version chains (paper Sec. 3.1, 3.3).  Shared by forward and backward.
static int run_prep(const Plan& p, void* ws, const void* q, const void* k, const void* w, cudaStream_t st) {
    const int d = p.d, nch = p.S * p.N;
    const long dd = (long)d * d;
    float* Dy = at<float>(ws, p.Dy);
    __nv_bfloat16* Qv16 = at<__nv_bfloat16>(ws, p.Qv16); __nv_bfloat16* Kv16 = at<__nv_bfloat16>(ws, p.Kv16);

    // fused per-chunk kernel: UT transform, boundary-adjusted tiles (version slot 0), chunk products (Dy level 0)
    {
        PrepTensorMaps tm;
        const uint64_t rows = (uint64_t)p.S * p.Lp;
        if (!(make_map(&tm.w, w, rows, d) && make_map(&tm.q, q, rows, d) && make_map(&tm.k, k, rows, d))) {
            g_last_cuda_error = (int)cudaErrorUnknown;
            return PATH_ERR_LAUNCH;
        }
        PrepParams pp{};
        pp.beta = at<float>(ws, p.betap);
        pp.q = (const __nv_bfloat16*)q; pp.k = (const __nv_bfloat16*)k;
        pp.ql = Qv16; pp.kr = Kv16;
        pp.Xqn = at<__nv_bfloat16>(ws, p.Xqn); pp.Yt = at<__nv_bfloat16>(ws, p.Yt);
        pp.P = Dy;
        if (p.bwd) {
            pp.Gm = at<float>(ws, p.Gm); pp.Ai = at<float>(ws, p.Ai); pp.Tt = at<float>(ws, p.Tt);
            pp.Xq = at<float>(ws, p.Xq); pp.Xk = at<float>(ws, p.Xk); pp.Y = at<float>(ws, p.Y);
            pp.U = at<float>(ws, p.U);
        }
        pp.status = at<uint32_t>(ws, p.status);
        LAUNCH(launch_chunk_prep(tm, pp, d, p.bwd, nch, st));
    }
    // dyadic run products Dy[l+1][b] = Dy[l][2b+1] Dy[l][2b]
    for (int l = 0; l + 1 <= p.nlev - 2; ++l) {
        const int cnt = p.N >> l, cnt2 = p.N >> (l + 1);
        const float* src = Dy + p.lv.dy_off[l];
        GemmProblem g = gemm_problem(Operand{src + dd, d, 1, 1}, Operand{src, 1, d, 1}, d, d, d);
        g.C = Dy + p.lv.dy_off[l + 1]; g.c_f32 = 1; g.ldc = d;
        AffineBatch ab{};
        ab.nb1 = cnt2;
        ab.a0 = (long)cnt * dd; ab.a1 = 2 * dd; ab.b0 = ab.a0; ab.b1 = ab.a1;
        ab.c0 = (long)cnt2 * dd; ab.c1 = dd;
        LAUNCH(launch_gemm(g, ab, p.S * cnt2, st));
    }
    // version chains
    for (int l2 = 1; l2 < p.nlev; ++l2) {
        for (int is_key = 0; is_key < 2; ++is_key) {
            VersionBatch v{};
            v.is_key = is_key; v.mode = 0; v.l2 = l2; v.S = p.S; v.N = p.N; v.Lp = p.Lp; v.d = d; v.lv = p.lv;
            v.xv = is_key ? Kv16 : Qv16; v.out16 = is_key ? Kv16 : Qv16;
            v.dy = Dy;
            LAUNCH(launch_gemm_version(v, st));
        }
    }
    return PATH_OK;
}

static int check_arch() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PATH_ERR_LAUNCH;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return PATH_ERR_LAUNCH;
    return major == 10 ? PATH_OK : PATH_ERR_ARCH;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// Pads q, k, v, w (ragged L) and beta into the workspace; returns the pointers the kernels should read.
static int stage_inputs(const Plan& p, void* ws, const void*& q, const void*& k, const void*& v, const void*& w,
                        const float* beta, const float* log_f, cudaStream_t st) {
    if (p.ragged) {
        LAUNCH(launch_pad_rows(q, at<void>(ws, p.qp), p.S, p.L, p.Lp, p.d, 0, st)); q = at<void>(ws, p.qp);
        LAUNCH(launch_pad_rows(k, at<void>(ws, p.kp), p.S, p.L, p.Lp, p.d, 0, st)); k = at<void>(ws, p.kp);
        LAUNCH(launch_pad_rows(v, at<void>(ws, p.vp), p.S, p.L, p.Lp, p.d, 0, st)); v = at<void>(ws, p.vp);
        LAUNCH(launch_pad_rows(w, at<void>(ws, p.wp), p.S, p.L, p.Lp, p.d, 0, st)); w = at<void>(ws, p.wp);
    }
    LAUNCH(launch_pad_vec(beta, at<float>(ws, p.betap), p.S, p.L, p.Lp, st));
    if (log_f) LAUNCH(launch_gate_prefix(log_f, at<float>(ws, p.G), p.S, p.L, p.Lp, st));
    return PATH_OK;
}

}  // namespace path

namespace path {

// Per-chunk chain rule through the UT transform and the boundary-adjusted tiles (no counterpart in the paper):
// from dQleft, dKright, dSd (diagonal logits), dP (chunk product) back to dq, dk, dw, dbeta.
static int run_chunk_chain(const Plan& p, void* ws, const void* q, const void* k, const void* w, void* dq, void* dk,
                           void* dw, float* dbeta, float scale, cudaStream_t st) {
    const int d = p.d, nch = p.S * p.N;
    const long Bd = (long)CHUNK * d, BB = (long)CHUNK * CHUNK, dd = (long)d * d;
    float* Gm = at<float>(ws, p.Gm); float* Tt = at<float>(ws, p.Tt); float* U = at<float>(ws, p.U);
    float* Ai = at<float>(ws, p.Ai); float* Xq = at<float>(ws, p.Xq); float* Xk = at<float>(ws, p.Xk);
    float* Y = at<float>(ws, p.Y);
    float* dQl = at<float>(ws, p.dQv); float* dKr = at<float>(ws, p.dKv);  // slot 0 of the version gradients
    float* dSd = at<float>(ws, p.dSd); float* dP = at<float>(ws, p.dDy);  // level 0 of the run-product gradients
    float* dXq = at<float>(ws, p.dXq); float* dY = at<float>(ws, p.dY); float* dT = at<float>(ws, p.dT);
    float* dXk = at<float>(ws, p.dXk); float* tmp = at<float>(ws, p.tmpBB); float* dA = at<float>(ws, p.dA);
    float* dU = at<float>(ws, p.dU); float* tq = at<float>(ws, p.tq); float* tk = at<float>(ws, p.tk);
    float* tw = at<float>(ws, p.tw); float* t1 = at<float>(ws, p.t1);
    const float* betap = at<float>(ws, p.betap);

    // operand shorthands: R = row-major as stored, T = transposed view
    auto R = [](const void* ptr, long ld, int f32) { return Operand{ptr, ld, 1, f32}; };   // A(m,k) = X[m][k]
    auto Tr = [](const void* ptr, long ld, int f32) { return Operand{ptr, 1, ld, f32}; };  // A(m,k) = X[k][m]
    // for the B operand B(k,n): Tr(X) means B(k,n) = X[k][n] (s_mn = 1, s_k = ld); R(X) means B(k,n) = X[n][k]
    auto run = [&](Operand A, long sa, Operand B, long sb, int M, int N, int K, float* C, long sc, float alpha, int mask,
                   int acc, const float* D = nullptr, long sd = 0, void* C2 = nullptr) -> int {
        GemmProblem g = gemm_problem(A, B, M, N, K);
        g.C = C; g.c_f32 = 1; g.ldc = N; g.alpha = alpha; g.mask = mask; g.accumulate = acc;
        if (D) { g.D = D; g.d_f32 = 1; g.ldd = N; }
        AffineBatch ab{};
        if (C2) {
            g.C2 = C2; g.ldc2 = N;
            ab.nb1 = p.N; ab.rows_total = p.L;
            ab.a0 = sa * p.N; ab.a1 = sa; ab.b0 = sb * p.N; ab.b1 = sb; ab.c0 = sc * p.N; ab.c1 = sc;
            ab.d0 = sd * p.N; ab.d1 = sd; ab.c20 = (long)p.L * d; ab.c21 = Bd;
        } else {
            ab = chunk_batch(p, sa, sb, sc, 0, sd);
        }
        LAUNCH(launch_gemm(g, ab, nch, st));
        return PATH_OK;
    };
#define RUN(...) do { int rc__ = run(__VA_ARGS__); if (rc__ != PATH_OK) return rc__; } while (0)
    const int B = CHUNK;
    // dSd below is the unscaled lower(dS) of the diagonal chunk; `scale` enters through the alphas.
    // dXq = lower(-dQl U^T - scale dSd Y^T)
    RUN(R(dQl, d, 1), Bd, R(U, d, 1), Bd, B, B, d, dXq, BB, -1.f, MASK_LOWER, ACC_NONE);
    RUN(R(dSd, B, 1), BB, R(Y, B, 1), BB, B, B, B, dXq, BB, -scale, MASK_LOWER, ACC_ADD);
    // dU = -Xq^T dQl - W dP
    RUN(Tr(Xq, B, 1), BB, Tr(dQl, d, 1), Bd, B, d, B, dU, Bd, -1.f, MASK_NONE, ACC_NONE);
    RUN(R(w, d, 0), Bd, Tr(dP, d, 1), dd, B, d, d, dU, Bd, -1.f, MASK_NONE, ACC_ADD);
    // dY = -W dKr^T - Xq^T dSd
    RUN(R(w, d, 0), Bd, R(dKr, d, 1), Bd, B, B, d, dY, BB, -1.f, MASK_NONE, ACC_NONE);
    RUN(Tr(Xq, B, 1), BB, Tr(dSd, B, 1), BB, B, B, B, dY, BB, -scale, MASK_NONE, ACC_ADD);
    // dT = lower(dY Xk^T + dU W^T)
    RUN(R(dY, B, 1), BB, R(Xk, B, 1), BB, B, B, B, dT, BB, 1.f, MASK_LOWER, ACC_NONE);
    RUN(R(dU, d, 1), Bd, R(w, d, 0), Bd, B, B, d, dT, BB, 1.f, MASK_LOWER, ACC_ADD);
    // dXk = strictLower(T~^T dY)
    RUN(Tr(Tt, B, 1), BB, Tr(dY, B, 1), BB, B, B, B, dXk, BB, 1.f, MASK_STRICT, ACC_NONE);
    // dbeta (first term) and dT <- dT D;  dA = strictLower(-Ainv^T (dT D) Ainv^T)
    LAUNCH(launch_beta_cols(Ai, dT, betap, t1, nch, st));
    RUN(Tr(Ai, B, 1), BB, Tr(dT, B, 1), BB, B, B, B, tmp, BB, 1.f, MASK_NONE, ACC_NONE);
    RUN(R(tmp, B, 1), BB, R(Ai, B, 1), BB, B, B, B, dA, BB, -1.f, MASK_STRICT, ACC_NONE);
    // dbeta (second term, final) and dA <- D dA = dGm
    LAUNCH(launch_beta_rows(dA, Gm, betap, t1, dbeta, p.S, p.N, p.L, st));
    // dq = dQl + dSd K + dXq W
    RUN(R(dSd, B, 1), BB, Tr(k, d, 0), Bd, B, d, B, tq, Bd, scale, MASK_NONE, ACC_NONE, dQl, Bd);
    RUN(R(dXq, B, 1), BB, Tr(w, d, 0), Bd, B, d, B, tq, Bd, 1.f, MASK_NONE, ACC_ADD, nullptr, 0, dq);
    // dk = dKr + dSd^T Q + dXk^T W
    RUN(Tr(dSd, B, 1), BB, Tr(q, d, 0), Bd, B, d, B, tk, Bd, scale, MASK_NONE, ACC_NONE, dKr, Bd);
    RUN(Tr(dXk, B, 1), BB, Tr(w, d, 0), Bd, B, d, B, tk, Bd, 1.f, MASK_NONE, ACC_ADD, nullptr, 0, dk);
    // dw = -Y dKr - U dP^T + T~^T dU + dXq^T Q + dXk K + dGm W + dGm^T W
    RUN(R(Y, B, 1), BB, Tr(dKr, d, 1), Bd, B, d, B, tw, Bd, -1.f, MASK_NONE, ACC_NONE);
    RUN(R(U, d, 1), Bd, R(dP, d, 1), dd, B, d, d, tw, Bd, -1.f, MASK_NONE, ACC_ADD);
    RUN(Tr(Tt, B, 1), BB, Tr(dU, d, 1), Bd, B, d, B, tw, Bd, 1.f, MASK_NONE, ACC_ADD);
    RUN(Tr(dXq, B, 1), BB, Tr(q, d, 0), Bd, B, d, B, tw, Bd, 1.f, MASK_NONE, ACC_ADD);
    RUN(R(dXk, B, 1), BB, Tr(k, d, 0), Bd, B, d, B, tw, Bd, 1.f, MASK_NONE, ACC_ADD);
    RUN(R(dA, B, 1), BB, Tr(w, d, 0), Bd, B, d, B, tw, Bd, 1.f, MASK_NONE, ACC_ADD);
    RUN(Tr(dA, B, 1), BB, Tr(w, d, 0), Bd, B, d, B, tw, Bd, 1.f, MASK_NONE, ACC_ADD, nullptr, 0, dw);
#undef RUN
    return PATH_OK;
}

static int run_backward(const Plan& p, void* ws, const void* q, const void* k, const void* v, const void* w,
                        const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, void* dw,
                        float* dbeta, float* dlog_f, float scale, cudaStream_t st) {
    const int d = p.d;
    const long dd = (long)d * d;
    const size_t SLd = (size_t)p.S * p.Lp * d;
    float* Dy = at<float>(ws, p.Dy); float* dDy = at<float>(ws, p.dDy);
    float* dQv = at<float>(ws, p.dQv); float* dKv = at<float>(ws, p.dKv);

    prof_mark(STG_ROWSTATS, 0, st);
    LAUNCH(launch_rowstats(o, d_o, lse, at<float>(ws, p.delta), at<float>(ws, p.lse2), p.S, p.L, p.Lp, d, st));
    const void* dop = d_o;
    if (p.ragged) {
        LAUNCH(launch_pad_rows(d_o, at<void>(ws, p.dop), p.S, p.L, p.Lp, d, 0, st));
        dop = at<void>(ws, p.dop);
    }
    CK(cudaMemsetAsync(dQv, 0, SLd * 4 * p.nslot, st));
    CK(cudaMemsetAsync(dKv, 0, SLd * 4 * p.nslot, st));
    CK(cudaMemsetAsync(dDy, 0, p.dy_bytes, st));
    if (p.gate) CK(cudaMemsetAsync(at<float>(ws, p.dGrow), 0, (size_t)p.S * p.Lp * 4, st));

    BwdTensorMaps tm;
    const uint64_t rows = (uint64_t)p.S * p.Lp;
    bool ok = make_map(&tm.q_raw, q, rows, d) && make_map(&tm.k_raw, k, rows, d) && make_map(&tm.v, v, rows, d) &&
              make_map(&tm.qv, at<void>(ws, p.Qv16), rows * p.nslot, d) &&
              make_map(&tm.kv, at<void>(ws, p.Kv16), rows * p.nslot, d) &&
              make_map(&tm.xqn, at<void>(ws, p.Xqn), rows, CHUNK) && make_map(&tm.yt, at<void>(ws, p.Yt), rows, CHUNK) &&
              make_map(&tm.d_o, dop, rows, d);
    if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
    BwdParams bp{};
    bp.dqv = dQv; bp.dkv = dKv; bp.dv = dv; bp.dsd = at<float>(ws, p.dSd); bp.dG = at<float>(ws, p.dG); bp.dGrow = at<float>(ws, p.dGrow);
    bp.lse2 = at<float>(ws, p.lse2); bp.delta = at<float>(ws, p.delta);
    bp.G = p.gate ? at<float>(ws, p.G) : nullptr;
    bp.status = at<uint32_t>(ws, p.status);
    bp.S = p.S; bp.L = p.L; bp.Lp = p.Lp; bp.N = p.N; bp.scale = scale;
    prof_mark(STG_ROWSTATS, 1, st);
    prof_mark(STG_FA_DKV, 0, st);
    LAUNCH(launch_fa_bwd(tm, bp, d, 0, st));
    prof_mark(STG_FA_DKV, 1, st);
    prof_mark(STG_FA_DQ, 0, st);
    LAUNCH(launch_fa_bwd(tm, bp, d, 1, st));
    prof_mark(STG_FA_DQ, 1, st);
    prof_mark(STG_CHAINS, 0, st);

    // version chains, top level first: gradients of the run products, then of the lower versions
    for (int l2 = p.nlev - 1; l2 >= 1; --l2)
        for (int is_key = 0; is_key < 2; ++is_key)
            for (int mode = 2; mode >= 1; --mode) {
                VersionBatch vb{};
                vb.is_key = is_key; vb.mode = mode; vb.l2 = l2; vb.S = p.S; vb.N = p.N; vb.Lp = p.Lp; vb.d = d;
                vb.lv = p.lv;
                vb.xv = is_key ? at<__nv_bfloat16>(ws, p.Kv16) : at<__nv_bfloat16>(ws, p.Qv16);
                vb.dxv = is_key ? dKv : dQv;
                vb.dy = Dy; vb.ddy = dDy;
                LAUNCH(launch_gemm_version(vb, st));
            }
    // run products, top-down: Dy[l][b] = Dy[l-1][2b+1] Dy[l-1][2b]
    for (int l = p.nlev - 2; l >= 1; --l) {
        const int cnt = p.N >> l, cntl = p.N >> (l - 1);
        const float* lo = Dy + p.lv.dy_off[l - 1];
        float* dlo = dDy + p.lv.dy_off[l - 1];
        const float* dup = dDy + p.lv.dy_off[l];
        AffineBatch ab{};
        ab.nb1 = cnt;
        ab.a0 = (long)cnt * dd; ab.a1 = dd;
        ab.b0 = (long)cntl * dd; ab.b1 = 2 * dd;
        ab.c0 = (long)cntl * dd; ab.c1 = 2 * dd;
        {   // d(left factor, index 2b+1) += dUp * (right factor)^T
            GemmProblem g = gemm_problem(Operand{dup, d, 1, 1}, Operand{lo, d, 1, 1}, d, d, d);
            g.C = dlo + dd; g.c_f32 = 1; g.ldc = d; g.accumulate = ACC_ADD;
            LAUNCH(launch_gemm(g, ab, p.S * cnt, st));
        }
        {   // d(right factor, index 2b) += (left factor)^T * dUp
            AffineBatch ab2 = ab;
            ab2.a0 = ab.b0; ab2.a1 = ab.b1; ab2.b0 = ab.a0; ab2.b1 = ab.a1;
            GemmProblem g = gemm_problem(Operand{lo + dd, 1, d, 1}, Operand{dup, 1, d, 1}, d, d, d);
            g.C = dlo; g.c_f32 = 1; g.ldc = d; g.accumulate = ACC_ADD;
            LAUNCH(launch_gemm(g, ab2, p.S * cnt, st));
        }
    }
    int rc = run_chunk_chain(p, ws, q, k, w, dq, dk, dw, dbeta, scale, st);
    if (rc != PATH_OK) return rc;
    if (dlog_f) {
        LAUNCH(launch_dsd_rowsum(at<float>(ws, p.dSd), at<float>(ws, p.dGdiag), p.S * p.N, st));
        LAUNCH(launch_gate_suffix(at<float>(ws, p.dG), at<float>(ws, p.dGrow), at<float>(ws, p.dGdiag), dlog_f, p.S, p.L,
                                  p.Lp, st));
    }
    prof_mark(STG_CHAINS, 1, st);
    return PATH_OK;
}

}  // namespace path

using namespace path;

extern "C" {

size_t path_attn_workspace_bytes(int B, int H, int L, int d, path_dtype_t dt, int has_gate, int for_backward) {
    Plan p;
    if (!make_plan(B, H, L, d, (int)dt, has_gate ? 1 : 0, for_backward ? 1 : 0, p)) return 0;
    return p.total;
}

int path_attn_fwd(const void* q, const void* k, const void* v, const void* w, const float* beta, const float* log_f,
                  void* o, float* lse, int B, int H, int L, int d, float scale, path_dtype_t dt, void* workspace,
                  size_t workspace_bytes, void* cuda_stream) {
    g_launches = 0;
    if (!q || !k || !v || !w || !beta || !o || !lse || !workspace) return PATH_ERR_NULL;
    Plan p;
    if (dt != PATH_BF16 && dt != PATH_FP32) return PATH_ERR_DTYPE;
    if (!make_plan(B, H, L, d, (int)dt, log_f ? 1 : 0, 0, p)) return PATH_ERR_SHAPE;
    if (dt != PATH_BF16) return PATH_ERR_DTYPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(w) || !aligned16(beta) || !aligned16(o) ||
        !aligned16(lse) || (log_f && !aligned16(log_f)) || ((uintptr_t)workspace & 255))
        return PATH_ERR_ALIGN;
    if (workspace_bytes < p.total) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, 256, st));

    prof_reset(STG_PREP, STG_PREP_BWD);
    prof_mark(STG_PREP, 0, st);
    rc = stage_inputs(p, workspace, q, k, v, w, beta, log_f, st);
    if (rc != PATH_OK) return rc;
    rc = run_prep(p, workspace, q, k, w, st);
    if (rc != PATH_OK) return rc;
    prof_mark(STG_PREP, 1, st);

    FwdTensorMaps tm;
    const uint64_t rows = (uint64_t)p.S * p.Lp;
    bool ok = make_map(&tm.q_raw, q, rows, d) && make_map(&tm.k_raw, k, rows, d) && make_map(&tm.v, v, rows, d) &&
              make_map(&tm.qv, at<void>(workspace, p.Qv16), rows * p.nslot, d) &&
              make_map(&tm.kv, at<void>(workspace, p.Kv16), rows * p.nslot, d) &&
              make_map(&tm.xqn, at<void>(workspace, p.Xqn), rows, CHUNK) &&
              make_map(&tm.yt, at<void>(workspace, p.Yt), rows, CHUNK);
    if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
    FwdParams fp{};
    fp.o = o; fp.lse = lse; fp.G = log_f ? at<float>(workspace, p.G) : nullptr;
    fp.status = at<uint32_t>(workspace, p.status);
    fp.S = p.S; fp.L = L; fp.Lp = p.Lp; fp.N = p.N; fp.scale = scale; fp.out_fp32 = 0;
    prof_mark(STG_FA_FWD, 0, st);
    LAUNCH(launch_fa_fwd(tm, fp, d, st));
    prof_mark(STG_FA_FWD, 1, st);
    return PATH_OK;
}

int path_attn_bwd(const void* q, const void* k, const void* v, const void* w, const float* beta, const float* log_f,
                  const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, void* dw,
                  float* dbeta, float* dlog_f, int B, int H, int L, int d, float scale, path_dtype_t dt,
                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
    g_launches = 0;
    if (!q || !k || !v || !w || !beta || !o || !lse || !d_o || !dq || !dk || !dv || !dw || !dbeta || !workspace)
        return PATH_ERR_NULL;
    if ((log_f == nullptr) != (dlog_f == nullptr)) return PATH_ERR_NULL;
    if (dt != PATH_BF16 && dt != PATH_FP32) return PATH_ERR_DTYPE;
    Plan p;
    if (!make_plan(B, H, L, d, (int)dt, log_f ? 1 : 0, 1, p)) return PATH_ERR_SHAPE;
    if (dt != PATH_BF16) return PATH_ERR_DTYPE;
    const void* ptrs[] = {q, k, v, w, beta, log_f, o, lse, d_o, dq, dk, dv, dw, dbeta, dlog_f};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return PATH_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return PATH_ERR_ALIGN;
    if (workspace_bytes < p.total) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, 256, st));
    prof_reset(STG_PREP_BWD, STG_COUNT);
    prof_mark(STG_PREP_BWD, 0, st);
    rc = stage_inputs(p, workspace, q, k, v, w, beta, log_f, st);
    if (rc != PATH_OK) return rc;
    rc = run_prep(p, workspace, q, k, w, st);
    if (rc != PATH_OK) return rc;
    prof_mark(STG_PREP_BWD, 1, st);
    return run_backward(p, workspace, q, k, v, w, o, lse, d_o, dq, dk, dv, dw, dbeta, dlog_f, scale, st);
}

int path_attn_device_status(const void* workspace, void* cuda_stream, unsigned int* detail) {
    if (!workspace) return PATH_ERR_NULL;
    unsigned int word = 0;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        g_last_cuda_error = (int)cudaGetLastError();
        return PATH_ERR_LAUNCH;
    }
    if (detail) *detail = word;
    return word == 0 ? PATH_OK : PATH_ERR_TIMEOUT;
}

const char* path_attn_strerror(int status) {
    switch (status) {
        case PATH_OK: return "ok";
        case PATH_ERR_NULL: return "a required pointer is NULL (or log_f / dlog_f not given together)";
        case PATH_ERR_SHAPE: return "unsupported shape (d must be 64 or 128; B, H, L >= 1)";
        case PATH_ERR_DTYPE: return "unsupported dtype for this entry point";
        case PATH_ERR_ALIGN: return "pointer not 16-byte aligned (workspace: 256-byte)";
        case PATH_ERR_WORKSPACE: return "workspace too small";
        case PATH_ERR_ARCH: return "device is not compute capability 10.x";
        case PATH_ERR_LAUNCH: return "a CUDA call failed";
        case PATH_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        default: return "unknown status";
    }
}

int path_attn_profile_enable(int on) {
    g_prof.on = on != 0;
    if (!on) prof_reset();
    return PATH_OK;
}

int path_attn_profile_read(float* ms, int n) {
    if (!ms) return PATH_ERR_NULL;
    int written = 0;
    for (int i = 0; i < STG_COUNT && i < n; ++i, ++written) {
        ms[i] = -1.f;
        if (!g_prof.on || !g_prof.created || !g_prof.used[i]) continue;
        if (cudaEventSynchronize(g_prof.ev[2 * i + 1]) != cudaSuccess ||
            cudaEventElapsedTime(&ms[i], g_prof.ev[2 * i], g_prof.ev[2 * i + 1]) != cudaSuccess) {
            g_last_cuda_error = (int)cudaGetLastError();
            return PATH_ERR_LAUNCH;
        }
    }
    return written;
}

const char* path_attn_profile_stage_name(int i) { return (i >= 0 && i < STG_COUNT) ? kStageNames[i] : ""; }

int path_attn_last_cuda_error(void) { return g_last_cuda_error; }
int path_attn_last_launch_count(void) { return g_launches; }

}  // extern "C"
