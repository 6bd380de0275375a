// C-ABI entry points of the PaTH attention library: argument validation, workspace planning, tensor-map
// encoding and the launch sequence.  All arithmetic runs in the kernels of linear.cu / fa_fwd.cu / fa_bwd.cu.
#include "../../include/path_attn.h"

#include <cstdio>
#include <cstring>
#include <mutex>

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

// Status block (the first 256 bytes of a workspace): word 0 = device status; bytes 32..47 = {kept, all} chunk pairs of the
// last gated forward (two 64-bit counters).
constexpr size_t kSkipCounterOffset = 32;

// ------------------------------------------------------------------------------------------- stage timing
// Optional per-thread instrumentation: CUDA events around groups of launches of the most recent call.
enum Stage { STG_PREP = 0, STG_LEVELS, STG_FA_FWD, STG_PREP_BWD, STG_LEVELS_BWDPREP, STG_ROWSTATS, STG_FA_DKV, STG_FA_DQ,
             STG_LEVELS_BWD, STG_CHAIN, STG_GATE, STG_COUNT };
static const char* const kStageNames[STG_COUNT] = {"chunk_prep", "levels_fwd", "fa_fwd", "bwd_chunk_prep", "bwd_levels_fwd",
                                                   "rowstats", "fa_bwd_dkv", "fa_bwd_dq", "bwd_levels", "bwd_chunk_chain",
                                                   "bwd_gate"};
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

// ------------------------------------------------------------------------------------------- forward state reuse
// A forward that ran on a backward-sized workspace leaves the chunk preparation (with the tiles the chain rule needs)
// in it, and ends by writing a record of the problem into the status block.  path_attn_bwd_reuse, the explicit request
// to skip the preparation, compares that record on the device before its first kernel reads the state; nothing is
// remembered on the host.
static StateRecord make_record(const void* q, const void* k, const void* v, const void* w, const float* beta,
                               const float* log_f, int B, int H, int L, int d, float scale) {
    StateRecord r{};
    r.magic = kStateMagic;
    r.q = q; r.k = k; r.v = v; r.w = w; r.beta = beta; r.log_f = log_f;
    r.B = B; r.H = H; r.L = L; r.d = d; r.scale = scale; r.gate = log_f ? 1 : 0;
    return r;
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

// bf16 matrix [rows][cols], box = [box_rows][64 cols], 128-byte swizzle (the low-rank layer's operands).
static bool make_map_box(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ------------------------------------------------------------------------------------------- workspace plan
struct Plan {
    int S, L, Lp, N, d, nlev, gate, bwd, ragged;
    LevelTable lv;
    VerLayout vl;
    uint64_t rows_q, rows_k;   // rows (of d elements) of the query / key version buffers
    size_t total;
    // offsets (bytes)
    size_t status, qp, kp, vp, wp, betap, G, tstats, nkeep, nvisit, Dyh, Dyl, Xqn, Yt, Qv16, Kv16;
    // backward only
    size_t dop, delta, lse2, dQv, dKv, dSd, dSdT, dG, dGrow, dGdiag, dDy;
    size_t sTh, sTl, sAh, sAl, sXk, sU;   // bf16 tiles kept by the chunk preparation for the chain rule
    size_t dy_bytes, dy_mats;
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
    p.vl = make_ver_layout(p.S, p.N, p.Lp, p.nlev);
    p.rows_q = (uint64_t)S * Lp + (uint64_t)S * p.vl.eq * CHUNK;
    p.rows_k = (uint64_t)S * Lp + (uint64_t)S * p.vl.ek * CHUNK;
    p.ragged = (L != p.Lp);
    size_t cur = 0;
    const size_t SLd = (size_t)S * Lp * d, SL = (size_t)S * Lp, SNBB = (size_t)S * p.N * CHUNK * CHUNK;
    p.status = bump(cur, 256);
    if (dt == PATH_FP32) {   // float32 tensors: forward only, computed from the definition; needs the gate prefix alone
        if (bwd) return false;
        p.G = bump(cur, gate ? SL * 4 : 0);
        p.total = cur;
        return true;
    }
    if (p.ragged) {
        p.qp = bump(cur, SLd * 2); p.kp = bump(cur, SLd * 2); p.vp = bump(cur, SLd * 2); p.wp = bump(cur, SLd * 2);
    }
    p.betap = bump(cur, SL * 4);
    if (gate) {
        p.G = bump(cur, SL * 4);
        p.tstats = bump(cur, (size_t)S * p.N * 8 * 4);   // per-chunk bounds and the resulting key-chunk counts: block skipping
        p.nkeep = bump(cur, (size_t)S * p.N * 4);
        p.nvisit = bump(cur, (size_t)S * p.N * 4);
    }
    const size_t keep = bwd ? 1 : 0;   // bf16 intermediates of the chunk preparation, kept for the chain rule
    p.sTh = bump(cur, keep * SNBB * 2); p.sTl = bump(cur, keep * SNBB * 2);
    p.sAh = bump(cur, keep * SNBB * 2); p.sAl = bump(cur, keep * SNBB * 2);
    p.sXk = bump(cur, keep * SNBB * 2);
    p.sU = bump(cur, keep * SLd * 2);
    size_t dy_elems = 0;
    for (int l = 0; l < 20; ++l) {
        p.lv.dy_off[l] = (long)dy_elems;
        p.lv.dy_cnt[l] = p.N >> l;
        if (l == 0 || l <= p.nlev - 2) dy_elems += (size_t)S * (p.N >> l) * d * d;
    }
    p.Dyh = bump(cur, dy_elems * 2);
    p.Dyl = bump(cur, dy_elems * 2);
    p.dy_mats = dy_elems / ((size_t)d * d);
    p.Xqn = bump(cur, SL * CHUNK * 2);
    p.Yt = bump(cur, SL * CHUNK * 2);
    p.Qv16 = bump(cur, p.rows_q * d * 2);
    p.Kv16 = bump(cur, p.rows_k * d * 2);
    p.dy_bytes = dy_elems * 2;
    if (bwd) {
        if (p.ragged) p.dop = bump(cur, SLd * 2);
        p.delta = bump(cur, SL * 4); p.lse2 = bump(cur, SL * 4);
        p.dQv = bump(cur, p.rows_q * d * 2); p.dKv = bump(cur, p.rows_k * d * 2);   // bf16
        p.dSd = bump(cur, gate ? SNBB * 4 : 0); p.dSdT = bump(cur, SNBB * 2); p.dG = bump(cur, SL * 4);
        p.dGrow = bump(cur, gate ? SL * 4 : 0); p.dGdiag = bump(cur, gate ? SL * 4 : 0);
        // bf16, each matrix written once by the CTA that owns it.  The backward never reads the run products' low planes
        // (gradient products take single bf16 operands), so their gradients take that place.
        p.dDy = p.Dyl;
    }
    p.total = cur;
    return true;
}

template <class T>
static T* at(void* ws, size_t off) { return reinterpret_cast<T*>((char*)ws + off); }

static bool make_level_maps(const Plan& p, void* ws, LevelTensorMaps& tm) {
    memset(&tm, 0, sizeof(tm));
    return make_map(&tm.dyh, at<void>(ws, p.Dyh), (uint64_t)p.dy_mats * p.d, p.d) &&
           make_map(&tm.dyl, at<void>(ws, p.Dyl), (uint64_t)p.dy_mats * p.d, p.d) &&
           make_map(&tm.qv, at<void>(ws, p.Qv16), p.rows_q, p.d) && make_map(&tm.kv, at<void>(ws, p.Kv16), p.rows_k, p.d) &&
           (!p.bwd || (make_map(&tm.dqv, at<void>(ws, p.dQv), p.rows_q, p.d) && make_map(&tm.dkv, at<void>(ws, p.dKv), p.rows_k, p.d) &&
                       make_map(&tm.ddy, at<void>(ws, p.dDy), (uint64_t)p.dy_mats * p.d, p.d)));
}

static LevelParams level_params(const Plan& p, void* ws) {
    LevelParams lp{};
    lp.lv = p.lv; lp.vl = p.vl; lp.S = p.S; lp.N = p.N; lp.Lp = p.Lp; lp.nlev = p.nlev;
    lp.dyh = at<__nv_bfloat16>(ws, p.Dyh); lp.dyl = at<__nv_bfloat16>(ws, p.Dyl);
    lp.qv = at<__nv_bfloat16>(ws, p.Qv16); lp.kv = at<__nv_bfloat16>(ws, p.Kv16);
    if (p.bwd) {
        lp.dqv = at<__nv_bfloat16>(ws, p.dQv); lp.dkv = at<__nv_bfloat16>(ws, p.dKv); lp.ddy16 = at<__nv_bfloat16>(ws, p.dDy);
    }
    if (p.gate) { lp.nkeep = at<int>(ws, p.nkeep); lp.nvisit = at<int>(ws, p.nvisit); }   // block skipping (see run_gate_skip)
    lp.status = at<uint32_t>(ws, p.status);
    return lp;
}

// Gated problems: which chunk pairs the sweeps can leave out (counts per query chunk and per key chunk, three small
// kernels).  Runs before the chunk preparation: the version chains stop at the highest level a kept pair uses.
static int run_gate_skip(const Plan& p, void* ws, const void* q, const void* k, const void* w, float scale, cudaStream_t st) {
    CK(cudaMemsetAsync(at<uint8_t>(ws, p.status + kSkipCounterOffset), 0, 16, st));
    LAUNCH(launch_gate_skip(q, k, w, at<float>(ws, p.betap), at<float>(ws, p.G), at<float>(ws, p.tstats), at<int>(ws, p.nkeep),
                            at<int>(ws, p.nvisit), at<unsigned long long>(ws, p.status + kSkipCounterOffset), p.S, p.L, p.Lp,
                            p.d, scale, st));
    g_launches += 2;
    return PATH_OK;
}

// Chunk preparation + dyadic run products + version chains (paper Sec. 3.1, 3.3).  Shared by forward and backward.
static int run_prep(const Plan& p, void* ws, const void* q, const void* k, const void* w, bool in_backward,
                    cudaStream_t st, bool with_levels = true, bool keys_only = false) {
    const int d = p.d, nch = p.S * p.N;
    const int stg_prep = in_backward ? STG_PREP_BWD : STG_PREP, stg_lev = in_backward ? STG_LEVELS_BWDPREP : STG_LEVELS;
    // fused per-chunk kernel: UT transform, boundary-adjusted tiles (version slot 0), chunk products (level 0)
    {
        PrepTensorMaps tm{};
        const uint64_t rows = (uint64_t)p.S * p.Lp;
        if (!(make_map(&tm.w, w, rows, d) && make_map(&tm.q, q, rows, d) && make_map(&tm.k, k, rows, d))) {
            g_last_cuda_error = (int)cudaErrorUnknown;
            return PATH_ERR_LAUNCH;
        }
        typedef __nv_bfloat16 bf;
        PrepParams pp{};
        pp.beta = at<float>(ws, p.betap);
        pp.q = (const bf*)q; pp.k = (const bf*)k;
        pp.ql = at<bf>(ws, p.Qv16); pp.kr = at<bf>(ws, p.Kv16);
        pp.Xqn = at<bf>(ws, p.Xqn); pp.Yt = at<bf>(ws, p.Yt);
        pp.Ph = at<bf>(ws, p.Dyh); pp.Pl = at<bf>(ws, p.Dyl);
        if (p.bwd) {
            pp.sAh = at<bf>(ws, p.sAh); pp.sAl = at<bf>(ws, p.sAl);
            if (!(make_map(&tm.th, at<void>(ws, p.sTh), rows, CHUNK) && make_map(&tm.tl, at<void>(ws, p.sTl), rows, CHUNK) &&
                  make_map(&tm.xk, at<void>(ws, p.sXk), rows, CHUNK) && make_map(&tm.u, at<void>(ws, p.sU), rows, d))) {
                g_last_cuda_error = (int)cudaErrorUnknown;
                return PATH_ERR_LAUNCH;
            }
        }
        pp.status = at<uint32_t>(ws, p.status);
        prof_mark(stg_prep, 0, st);
        LAUNCH(launch_chunk_prep(tm, pp, d, keys_only ? PREP_KEYS : (p.bwd ? PREP_SAVE : PREP_FWD), nch, st));
        prof_mark(stg_prep, 1, st);
    }
    if (p.nlev < 2 || !with_levels) return PATH_OK;
    LevelTensorMaps tm;
    if (!make_level_maps(p, ws, tm)) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
    LevelParams lp = level_params(p, ws);
    prof_mark(stg_lev, 0, st);
    for (int l = 0; l + 1 <= p.nlev - 2;) {       // run products of 2, 4, ... chunks, up to three levels per launch
        const int left = p.nlev - 2 - l;
        lp.l = l;
        lp.fuse = left >= 3 ? 3 : left;
        LAUNCH(launch_level_kernel(lp.fuse >= 2 ? LEVEL_DYADIC_FUSED : LEVEL_DYADIC_FWD, tm, lp, d, st));
        l += lp.fuse;
    }
    lp.l = p.nlev;                                // query and key versions: one CTA per chunk walks its chain
    LAUNCH(launch_level_kernel(LEVEL_VERSION_FWD, tm, lp, d, st));
    prof_mark(stg_lev, 1, st);
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
// With run = false only the pointers are redirected (the padded copies are already in the workspace).
static int stage_inputs(const Plan& p, void* ws, const void*& q, const void*& k, const void*& v, const void*& w,
                        const float* beta, const float* log_f, bool run, cudaStream_t st) {
    if (p.ragged) {
        if (run) {
            LAUNCH(launch_pad_rows(q, at<void>(ws, p.qp), p.S, p.L, p.Lp, p.d, 0, st));
            LAUNCH(launch_pad_rows(k, at<void>(ws, p.kp), p.S, p.L, p.Lp, p.d, 0, st));
            LAUNCH(launch_pad_rows(v, at<void>(ws, p.vp), p.S, p.L, p.Lp, p.d, 0, st));
            LAUNCH(launch_pad_rows(w, at<void>(ws, p.wp), p.S, p.L, p.Lp, p.d, 0, st));
        }
        q = at<void>(ws, p.qp); k = at<void>(ws, p.kp); v = at<void>(ws, p.vp); w = at<void>(ws, p.wp);
    }
    if (run) {
        LAUNCH(launch_pad_vec(beta, at<float>(ws, p.betap), p.S, p.L, p.Lp, st));
        if (log_f) LAUNCH(launch_gate_prefix(log_f, at<float>(ws, p.G), p.S, p.L, p.Lp, st));
    }
    return PATH_OK;
}

}  // namespace path

namespace path {

// Per-chunk chain rule through the UT transform and the boundary-adjusted tiles: one fused kernel.
static int run_chunk_chain(const Plan& p, void* ws, const void* q, const void* k, const void* w, void* dq, void* dk,
                           void* dw, float* dbeta, float scale, cudaStream_t st) {
    const int d = p.d;
    const uint64_t rows = (uint64_t)p.S * p.Lp;
    ChainTensorMaps tm;
    bool ok = make_map(&tm.w, w, rows, d) && make_map(&tm.q, q, rows, d) && make_map(&tm.k, k, rows, d) &&
              make_map(&tm.u, at<void>(ws, p.sU), rows, d) && make_map(&tm.yt, at<void>(ws, p.Yt), rows, CHUNK) &&
              make_map(&tm.xqn, at<void>(ws, p.Xqn), rows, CHUNK) && make_map(&tm.xk, at<void>(ws, p.sXk), rows, CHUNK) &&
              make_map(&tm.th, at<void>(ws, p.sTh), rows, CHUNK) && make_map(&tm.tl, at<void>(ws, p.sTl), rows, CHUNK) &&
              make_map(&tm.ah, at<void>(ws, p.sAh), rows, CHUNK) && make_map(&tm.al, at<void>(ws, p.sAl), rows, CHUNK) &&
              make_map(&tm.dsdt, at<void>(ws, p.dSdT), (uint64_t)p.S * p.N * CHUNK, CHUNK) &&
              make_map(&tm.dql, at<void>(ws, p.dQv), rows, d) && make_map(&tm.dkr, at<void>(ws, p.dKv), rows, d) &&
              make_map(&tm.dp, at<void>(ws, p.dDy), (uint64_t)p.S * p.N * d, d);   // level 0 of the run-product gradients
    if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
    ChainParams cp{};
    cp.dql = at<__nv_bfloat16>(ws, p.dQv); cp.dkr = at<__nv_bfloat16>(ws, p.dKv);   // slot 0 of the version gradients: the final sums
    cp.beta = at<float>(ws, p.betap);
    cp.dq = (__nv_bfloat16*)dq; cp.dk = (__nv_bfloat16*)dk; cp.dw = (__nv_bfloat16*)dw; cp.dbeta = dbeta;
    cp.status = at<uint32_t>(ws, p.status);
    cp.N = p.N; cp.L = p.L; cp.scale = scale;
    LAUNCH(launch_chunk_chain(tm, cp, d, p.S * p.N, st));
    return PATH_OK;
}

static int run_backward(const Plan& p, void* ws, const void* q, const void* k, const void* v, const void* w,
                        const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, void* dw,
                        float* dbeta, float* dlog_f, float scale, cudaStream_t st) {
    const int d = p.d;
    __nv_bfloat16* dQv = at<__nv_bfloat16>(ws, p.dQv); __nv_bfloat16* dKv = at<__nv_bfloat16>(ws, p.dKv);

    prof_mark(STG_ROWSTATS, 0, st);
    LAUNCH(launch_rowstats(o, d_o, lse, p.gate ? at<float>(ws, p.G) : nullptr, at<float>(ws, p.delta), at<float>(ws, p.lse2),
                           p.S, p.L, p.Lp, d, st));
    const void* dop = d_o;
    if (p.ragged) {
        LAUNCH(launch_pad_rows(d_o, at<void>(ws, p.dop), p.S, p.L, p.Lp, d, 0, st));
        dop = at<void>(ws, p.dop);
    }
    if (p.gate) CK(cudaMemsetAsync(at<float>(ws, p.dGrow), 0, (size_t)p.S * p.Lp * 4, st));

    BwdTensorMaps tm;
    const uint64_t rows = (uint64_t)p.S * p.Lp;
    bool ok = make_map(&tm.q_raw, q, rows, d) && make_map(&tm.k_raw, k, rows, d) && make_map(&tm.v, v, rows, d) &&
              make_map(&tm.qv, at<void>(ws, p.Qv16), p.rows_q, d) &&
              make_map(&tm.kv, at<void>(ws, p.Kv16), p.rows_k, d) &&
              make_map(&tm.xqn, at<void>(ws, p.Xqn), rows, CHUNK) && make_map(&tm.yt, at<void>(ws, p.Yt), rows, CHUNK) &&
              make_map(&tm.d_o, dop, rows, d);
    if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
    BwdParams bp{};
    bp.dqv = dQv; bp.dkv = dKv; bp.dv = dv; bp.dsd = p.gate ? at<float>(ws, p.dSd) : nullptr; bp.dsdt = at<__nv_bfloat16>(ws, p.dSdT); bp.dG = at<float>(ws, p.dG); bp.dGrow = at<float>(ws, p.dGrow);
    bp.lse2 = at<float>(ws, p.lse2); bp.delta = at<float>(ws, p.delta);
    bp.G = p.gate ? at<float>(ws, p.G) : nullptr;
    bp.status = at<uint32_t>(ws, p.status);
    bp.S = p.S; bp.L = p.L; bp.Lp = p.Lp; bp.N = p.N; bp.scale = scale; bp.vl = p.vl;
    if (p.gate) { bp.nkeep = at<int>(ws, p.nkeep); bp.nvisit = at<int>(ws, p.nvisit); }   // block skipping: see run_gate_skip
    prof_mark(STG_ROWSTATS, 1, st);
    prof_mark(STG_FA_DKV, 0, st);
    LAUNCH(launch_fa_bwd(tm, bp, d, 0, st));
    prof_mark(STG_FA_DKV, 1, st);
    prof_mark(STG_FA_DQ, 0, st);
    LAUNCH(launch_fa_bwd(tm, bp, d, 1, st));
    prof_mark(STG_FA_DQ, 1, st);
    prof_mark(STG_LEVELS_BWD, 0, st);

    // version chains and run products, top level first: one launch per level finishes the gradients of that level's run
    // products and adds the chains' carries to the version gradients one level down (slot 0 ends up holding the final
    // sums the chunk chain rule loads; level 0 of the run-product gradients is its dP)
    {
        LevelTensorMaps ltm;
        if (!make_level_maps(p, ws, ltm)) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
        LevelParams lp = level_params(p, ws);
        for (int l = p.nlev - 2 > 0 ? p.nlev - 2 : 0; l >= 0; --l) {
            lp.l = l;
            LAUNCH(launch_level_kernel(LEVEL_BWD, ltm, lp, d, st));
        }
    }
    prof_mark(STG_LEVELS_BWD, 1, st);
    prof_mark(STG_CHAIN, 0, st);
    int rc = run_chunk_chain(p, ws, q, k, w, dq, dk, dw, dbeta, scale, st);
    if (rc != PATH_OK) return rc;
    prof_mark(STG_CHAIN, 1, st);
    prof_mark(STG_GATE, 0, st);
    if (dlog_f) {
        LAUNCH(launch_dsd_rowsum(at<float>(ws, p.dSd), at<float>(ws, p.dGdiag), p.S * p.N, st));
        LAUNCH(launch_gate_suffix(at<float>(ws, p.dG), at<float>(ws, p.dGrow), at<float>(ws, p.dGdiag), dlog_f, p.S, p.L,
                                  p.Lp, st));
    }
    prof_mark(STG_GATE, 1, st);
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
    if (dt == PATH_FP32) {
        if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(w) || !aligned16(beta) || !aligned16(o) ||
            !aligned16(lse) || (log_f && !aligned16(log_f)) || ((uintptr_t)workspace & 255))
            return PATH_ERR_ALIGN;
        if (workspace_bytes < p.total) return PATH_ERR_WORKSPACE;
        int rc32 = check_arch();
        if (rc32 != PATH_OK) return rc32;
        cudaStream_t st32 = (cudaStream_t)cuda_stream;
        CK(cudaMemsetAsync(workspace, 0, 256, st32));
        float* G = nullptr;
        if (log_f) {
            G = at<float>(workspace, p.G);
            LAUNCH(launch_gate_prefix(log_f, G, p.S, L, p.Lp, st32));
        }
        LAUNCH(launch_fp32_fwd((const float*)q, (const float*)k, (const float*)v, (const float*)w, beta, G, (float*)o, lse,
                               p.S, L, p.Lp, d, scale, st32));
        return PATH_OK;
    }
    // A workspace large enough for the backward gets the backward's layout: the chunk preparation then also keeps
    // the tiles the chain rule needs, and path_attn_bwd on the same workspace and inputs does not redo it.
    const StateRecord rec = make_record(q, k, v, w, beta, log_f, B, H, L, d, scale);   // (the caller's pointers, before padding)
    bool keep_state = false;
    {
        Plan pb;
        if (make_plan(B, H, L, d, (int)dt, log_f ? 1 : 0, 1, pb) && workspace_bytes >= pb.total) { p = pb; keep_state = true; }
    }
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(w) || !aligned16(beta) || !aligned16(o) ||
        !aligned16(lse) || (log_f && !aligned16(log_f)) || ((uintptr_t)workspace & 255))
        return PATH_ERR_ALIGN;
    if (workspace_bytes < p.total) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, 256, st));

    prof_reset(STG_PREP, STG_PREP_BWD);
    rc = stage_inputs(p, workspace, q, k, v, w, beta, log_f, true, st);
    if (rc != PATH_OK) return rc;
    if (log_f) {
        rc = run_gate_skip(p, workspace, q, k, w, scale, st);
        if (rc != PATH_OK) return rc;
    }
    rc = run_prep(p, workspace, q, k, w, false, st);
    if (rc != PATH_OK) return rc;

    FwdTensorMaps tm;
    const uint64_t rows = (uint64_t)p.S * p.Lp;
    bool ok = make_map(&tm.q_raw, q, rows, d) && make_map(&tm.k_raw, k, rows, d) && make_map(&tm.v, v, rows, d) &&
              make_map(&tm.qv, at<void>(workspace, p.Qv16), p.rows_q, d) &&
              make_map(&tm.kv, at<void>(workspace, p.Kv16), p.rows_k, d) &&
              make_map(&tm.xqn, at<void>(workspace, p.Xqn), rows, CHUNK) &&
              make_map(&tm.yt, at<void>(workspace, p.Yt), rows, CHUNK);
    if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
    FwdParams fp{};
    fp.o = o; fp.lse = lse; fp.G = log_f ? at<float>(workspace, p.G) : nullptr;
    fp.status = at<uint32_t>(workspace, p.status);
    fp.S = p.S; fp.L = L; fp.Lp = p.Lp; fp.N = p.N; fp.scale = scale; fp.out_fp32 = 0; fp.vl = p.vl;
    prof_mark(STG_FA_FWD, 0, st);
    if (log_f) fp.nkeep = at<int>(workspace, p.nkeep);   // block skipping: see run_gate_skip
    LAUNCH(launch_fa_fwd(tm, fp, d, st));
    prof_mark(STG_FA_FWD, 1, st);
    if (keep_state) LAUNCH(launch_state_write(at<void>(workspace, p.status + kStateRecordOffset), rec, st));
    return PATH_OK;
}

static int backward_entry(const void* q, const void* k, const void* v, const void* w, const float* beta, const float* log_f,
                          const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, void* dw,
                          float* dbeta, float* dlog_f, int B, int H, int L, int d, float scale, path_dtype_t dt,
                          void* workspace, size_t workspace_bytes, void* cuda_stream, bool reuse) {
    g_launches = 0;
    if (!q || !k || !v || !w || !beta || !o || !lse || !d_o || !dq || !dk || !dv || !dw || !dbeta || !workspace)
        return PATH_ERR_NULL;
    if ((log_f == nullptr) != (dlog_f == nullptr)) return PATH_ERR_NULL;
    if (dt != PATH_BF16 && dt != PATH_FP32) return PATH_ERR_DTYPE;
    Plan p;
    if (dt != PATH_BF16) return PATH_ERR_DTYPE;   // float32 tensors: forward only
    if (!make_plan(B, H, L, d, (int)dt, log_f ? 1 : 0, 1, p)) return PATH_ERR_SHAPE;
    const void* ptrs[] = {q, k, v, w, beta, log_f, o, lse, d_o, dq, dk, dv, dw, dbeta, dlog_f};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return PATH_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return PATH_ERR_ALIGN;
    if (workspace_bytes < p.total) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, kSkipCounterOffset, st));   // the status word; the block-skipping counters may be reused
    prof_reset(STG_PREP_BWD, STG_COUNT);
    if (reuse) {
        // the record the forward left must describe this very problem (for a gated one the scale too: the block-skipping
        // counts, and with them the levels the version chains were built up to, depend on it)
        LAUNCH(launch_state_check(at<void>(workspace, p.status + kStateRecordOffset),
                                  make_record(q, k, v, w, beta, log_f, B, H, L, d, scale), at<uint32_t>(workspace, p.status), st));
    } else {
        CK(cudaMemsetAsync(at<uint8_t>(workspace, p.status + kStateRecordOffset), 0, sizeof(StateRecord), st));
    }
    rc = stage_inputs(p, workspace, q, k, v, w, beta, log_f, !reuse, st);
    if (rc != PATH_OK) return rc;
    if (!reuse) {
        if (log_f) {
            rc = run_gate_skip(p, workspace, q, k, w, scale, st);
            if (rc != PATH_OK) return rc;
        }
        rc = run_prep(p, workspace, q, k, w, true, st);
        if (rc != PATH_OK) return rc;
    }
    return run_backward(p, workspace, q, k, v, w, o, lse, d_o, dq, dk, dv, dw, dbeta, dlog_f, scale, st);
}

int path_attn_bwd(const void* q, const void* k, const void* v, const void* w, const float* beta, const float* log_f,
                  const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, void* dw,
                  float* dbeta, float* dlog_f, int B, int H, int L, int d, float scale, path_dtype_t dt,
                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return backward_entry(q, k, v, w, beta, log_f, o, lse, d_o, dq, dk, dv, dw, dbeta, dlog_f, B, H, L, d, scale, dt,
                          workspace, workspace_bytes, cuda_stream, false);
}

int path_attn_bwd_reuse(const void* q, const void* k, const void* v, const void* w, const float* beta, const float* log_f,
                        const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, void* dw,
                        float* dbeta, float* dlog_f, int B, int H, int L, int d, float scale, path_dtype_t dt,
                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return backward_entry(q, k, v, w, beta, log_f, o, lse, d_o, dq, dk, dv, dw, dbeta, dlog_f, B, H, L, d, scale, dt,
                          workspace, workspace_bytes, cuda_stream, true);
}

int path_attn_selftest_timeout(void* workspace, unsigned int limit_us, void* cuda_stream) {
    g_launches = 0;
    if (!workspace) return PATH_ERR_NULL;
    if ((uintptr_t)workspace & 255) return PATH_ERR_ALIGN;
    if (limit_us < 1 || limit_us > 100000) return PATH_ERR_SHAPE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, 256, st));
    LAUNCH(launch_selftest_wait((uint32_t*)workspace, (long long)limit_us * 2000LL, st));   // ~2 clock ticks per ns
    return PATH_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------- forward without a workspace
// Scratch for path_attn_fwd_static lives in the library image: one buffer per device that loads the module.  In host
// code the array's name is only a handle; its device address is looked up once per device and cached here.
static __device__ __align__(256) unsigned char g_static_scratch[PATH_ATTN_STATIC_SCRATCH_BYTES];
static constexpr int kMaxDevices = 64;
static void* g_static_scratch_addr[kMaxDevices] = {};
static std::mutex g_static_scratch_mutex;

static int static_scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        path::g_last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorInvalidDevice);
        return PATH_ERR_LAUNCH;
    }
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* addr = nullptr;
        e = cudaGetSymbolAddress(&addr, g_static_scratch);   // resolves against the current device's copy
        if (e != cudaSuccess || addr == nullptr) {
            path::g_last_cuda_error = (int)(e != cudaSuccess ? e : cudaErrorInvalidSymbol);
            return PATH_ERR_LAUNCH;
        }
        g_static_scratch_addr[dev] = addr;
    }
    *out = g_static_scratch_addr[dev];
    return PATH_OK;
}

extern "C" {

int path_attn_fwd_static(const void* q, const void* k, const void* v, const void* w, const float* beta,
                         const float* log_f, void* o, float* lse, int B, int H, int L, int d, float scale,
                         path_dtype_t dt, void* cuda_stream, void** scratch_out) {
    if (dt != PATH_BF16 && dt != PATH_FP32) return PATH_ERR_DTYPE;
    const size_t need = path_attn_workspace_bytes(B, H, L, d, dt, log_f ? 1 : 0, 0);
    if (need == 0) return PATH_ERR_SHAPE;
    if (need > (size_t)PATH_ATTN_STATIC_SCRATCH_BYTES) return PATH_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != PATH_OK) return rc;
    const bool timing = path::g_prof.on;   // stage timing would create CUDA events on first use
    path::g_prof.on = false;
    // (the forward's own size, not the buffer's: a larger figure would select the backward's layout and keep its state)
    rc = path_attn_fwd(q, k, v, w, beta, log_f, o, lse, B, H, L, d, scale, dt, scratch, need, cuda_stream);
    path::g_prof.on = timing;
    if (scratch_out) *scratch_out = scratch;
    return rc;
}

// ------------------------------------------------------------------------------------------- context-parallel path
// Layouts of the two caller-owned buffers of the segment-level calls (paper Sec. 3.5); every part starts 256-byte aligned.
struct CpLayout {
    int S, L, Lp, N, d;
    size_t x, gq, o_acc, lse_acc, state_total;        // state: query tiles pulled back so far, their gate terms, running result
    size_t kend, v, pseg, gk, gtot, message_total;    // message: what a segment hands to the holders of later queries
    size_t o_t, lse_t, step_total;                    // scratch of one step (after the 256-byte status block)
};
static bool cp_layout(int B, int H, int L, int d, CpLayout& c) {
    Plan p;
    if (!make_plan(B, H, L, d, PATH_BF16, 0, 0, p)) return false;
    c.S = p.S; c.L = L; c.Lp = p.Lp; c.N = p.N; c.d = d;
    const size_t SLpd = (size_t)p.S * p.Lp * d, SLp = (size_t)p.S * p.Lp, SLd = (size_t)p.S * L * d, SL = (size_t)p.S * L;
    size_t cur = 0;
    c.x = bump(cur, SLpd * 2); c.gq = bump(cur, SLp * 4); c.o_acc = bump(cur, SLd * 4); c.lse_acc = bump(cur, SL * 4);
    c.state_total = cur;
    cur = 0;
    c.kend = bump(cur, SLpd * 2); c.v = bump(cur, SLpd * 2); c.pseg = bump(cur, (size_t)p.S * 2 * d * d * 2);
    c.gk = bump(cur, SLp * 4); c.gtot = bump(cur, (size_t)p.S * 4);
    c.message_total = cur;
    cur = 256;
    c.o_t = bump(cur, SLd * 4); c.lse_t = bump(cur, SL * 4);
    c.step_total = cur;
    return true;
}

size_t path_attn_cp_state_bytes(int B, int H, int L, int d) {
    CpLayout c;
    return cp_layout(B, H, L, d, c) ? c.state_total : 0;
}
size_t path_attn_cp_message_bytes(int B, int H, int L, int d) {
    CpLayout c;
    return cp_layout(B, H, L, d, c) ? c.message_total : 0;
}
size_t path_attn_cp_workspace_bytes(int B, int H, int L, int d, int has_gate) {
    CpLayout c;
    Plan p;
    if (!cp_layout(B, H, L, d, c) || !make_plan(B, H, L, d, PATH_BF16, has_gate ? 1 : 0, 0, p)) return 0;
    return p.total > c.step_total ? p.total : c.step_total;
}

int path_attn_cp_prepare(const void* q, const void* k, const void* v, const void* w, const float* beta, const float* log_f,
                         void* state, void* message, int B, int H, int L, int d, float scale, path_dtype_t dt,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
    g_launches = 0;
    if (!q || !k || !v || !w || !beta || !state || !message || !workspace) return PATH_ERR_NULL;
    if (dt != PATH_BF16) return PATH_ERR_DTYPE;
    Plan p;
    CpLayout c;
    if (!make_plan(B, H, L, d, (int)dt, log_f ? 1 : 0, 0, p) || !cp_layout(B, H, L, d, c)) return PATH_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(w) || !aligned16(beta) || (log_f && !aligned16(log_f)) ||
        ((uintptr_t)workspace & 255) || ((uintptr_t)state & 255) || ((uintptr_t)message & 255))
        return PATH_ERR_ALIGN;
    if (workspace_bytes < path_attn_cp_workspace_bytes(B, H, L, d, log_f ? 1 : 0)) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, 256, st));
    rc = stage_inputs(p, workspace, q, k, v, w, beta, log_f, true, st);
    if (rc != PATH_OK) return rc;
    if (log_f) {
        rc = run_gate_skip(p, workspace, q, k, w, scale, st);
        if (rc != PATH_OK) return rc;
    }
    rc = run_prep(p, workspace, q, k, w, false, st);
    if (rc != PATH_OK) return rc;
    // the segment's own (causal) attention, as a float32 running result
    {
        FwdTensorMaps tm;
        const uint64_t rows = (uint64_t)p.S * p.Lp;
        bool ok = make_map(&tm.q_raw, q, rows, d) && make_map(&tm.k_raw, k, rows, d) && make_map(&tm.v, v, rows, d) &&
                  make_map(&tm.qv, at<void>(workspace, p.Qv16), p.rows_q, d) &&
                  make_map(&tm.kv, at<void>(workspace, p.Kv16), p.rows_k, d) &&
                  make_map(&tm.xqn, at<void>(workspace, p.Xqn), rows, CHUNK) && make_map(&tm.yt, at<void>(workspace, p.Yt), rows, CHUNK);
        if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
        FwdParams fp{};
        fp.o = at<float>(state, c.o_acc); fp.lse = at<float>(state, c.lse_acc); fp.G = log_f ? at<float>(workspace, p.G) : nullptr;
        fp.status = at<uint32_t>(workspace, p.status);
        fp.S = p.S; fp.L = L; fp.Lp = p.Lp; fp.N = p.N; fp.scale = scale; fp.out_fp32 = 1; fp.vl = p.vl;
        if (log_f) fp.nkeep = at<int>(workspace, p.nkeep);
        LAUNCH(launch_fa_fwd(tm, fp, d, st));
    }
    // keys advanced to the segment's end, queries pulled back to its start, the product of the whole segment
    {
        LevelTensorMaps tm;
        if (!make_level_maps(p, workspace, tm)) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
        LevelParams lp = level_params(p, workspace);
        lp.L = p.Lp; lp.cap = p.Lp;   // (whole padded chunks: the padded rows of the prepared tiles are zero)
        lp.edge16 = at<__nv_bfloat16>(message, c.kend);
        LAUNCH(launch_level_kernel(LEVEL_KEY_CACHE, tm, lp, d, st));
        lp.edge16 = at<__nv_bfloat16>(state, c.x);
        lp.pseg = at<__nv_bfloat16>(message, c.pseg);
        LAUNCH(launch_level_kernel(LEVEL_QUERY_EDGE, tm, lp, d, st));
    }
    CK(cudaMemcpyAsync(at<void>(message, c.v), v, (size_t)p.S * p.Lp * d * 2, cudaMemcpyDeviceToDevice, st));
    LAUNCH(launch_cp_gate(log_f ? at<float>(workspace, p.G) : nullptr, at<float>(state, c.gq), at<float>(message, c.gk),
                          at<float>(message, c.gtot), p.S, L, p.Lp, st));
    return PATH_OK;
}

int path_attn_cp_step(void* state, const void* message, int B, int H, int Lq, int Lk, int d, float scale, void* workspace,
                      size_t workspace_bytes, void* cuda_stream) {
    g_launches = 0;
    if (!state || !message || !workspace) return PATH_ERR_NULL;
    CpLayout cq, ck;
    if (!cp_layout(B, H, Lq, d, cq) || !cp_layout(B, H, Lk, d, ck)) return PATH_ERR_SHAPE;
    if (((uintptr_t)workspace & 255) || ((uintptr_t)state & 255) || ((uintptr_t)message & 255)) return PATH_ERR_ALIGN;
    if (workspace_bytes < cq.step_total) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, 256, st));
    void* msg = const_cast<void*>(message);
    // every query chunk of this segment against every key chunk of the incoming one
    {
        FwdTensorMaps tm;
        bool ok = make_map(&tm.qv, at<void>(state, cq.x), (uint64_t)cq.S * cq.Lp, d) &&
                  make_map(&tm.kv, at<void>(msg, ck.kend), (uint64_t)ck.S * ck.Lp, d) &&
                  make_map(&tm.v, at<void>(msg, ck.v), (uint64_t)ck.S * ck.Lp, d);
        if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
        tm.q_raw = tm.k_raw = tm.xqn = tm.yt = tm.qv;   // unused by this sweep, but every descriptor gets prefetched
        FwdParams fp{};
        fp.o = at<float>(workspace, cq.o_t); fp.lse = at<float>(workspace, cq.lse_t);
        fp.G = at<float>(state, cq.gq); fp.Gk = at<float>(msg, ck.gk);
        fp.status = (uint32_t*)workspace;
        fp.S = cq.S; fp.L = Lq; fp.Lp = cq.Lp; fp.N = cq.N; fp.Nk = ck.N; fp.Lkp = ck.Lp; fp.scale = scale; fp.out_fp32 = 1;
        LAUNCH(launch_fa_fwd_cross(tm, fp, d, st));
    }
    LAUNCH(launch_cp_merge(at<float>(state, cq.o_acc), at<float>(state, cq.lse_acc), at<float>(workspace, cq.o_t),
                           at<float>(workspace, cq.lse_t), (size_t)cq.S * Lq, d, st));
    // the queries move on past the attended segment: x <- x P(segment), gate terms += the segment's total
    {
        LevelTensorMaps tm;
        memset(&tm, 0, sizeof(tm));
        bool ok = make_map(&tm.qv, at<void>(state, cq.x), (uint64_t)cq.S * cq.Lp, d) &&
                  make_map(&tm.dyh, at<void>(msg, ck.pseg), (uint64_t)ck.S * 2 * d, d);
        if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
        tm.dyl = tm.kv = tm.dqv = tm.dkv = tm.ddy = tm.qv;
        LevelParams lp{};
        lp.S = cq.S; lp.N = cq.N; lp.Lp = cq.Lp;
        lp.qv = at<__nv_bfloat16>(state, cq.x);
        lp.gq = at<float>(state, cq.gq); lp.gtot = at<float>(msg, ck.gtot);
        lp.status = (uint32_t*)workspace;
        LAUNCH(launch_level_kernel(LEVEL_APPLY_PRODUCT, tm, lp, d, st));
    }
    return PATH_OK;
}

int path_attn_cp_finish(const void* state, void* o, float* lse, int B, int H, int L, int d, void* cuda_stream) {
    g_launches = 0;
    if (!state || !o || !lse) return PATH_ERR_NULL;
    CpLayout c;
    if (!cp_layout(B, H, L, d, c)) return PATH_ERR_SHAPE;
    if (((uintptr_t)state & 255) || !aligned16(o) || !aligned16(lse)) return PATH_ERR_ALIGN;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    void* st_ = const_cast<void*>(state);
    LAUNCH(launch_cp_finish(at<float>(st_, c.o_acc), at<float>(st_, c.lse_acc), o, lse, (size_t)c.S * L, d, (cudaStream_t)cuda_stream));
    return PATH_OK;
}

int path_attn_prefill_cache(const void* k, const void* v, const void* w, const float* beta, const float* log_f, float* kc,
                            void* vc, float* gc, int B, int H, int L, int d, int cap, path_dtype_t dt, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
    g_launches = 0;
    if (!k || !v || !w || !beta || !kc || !vc || !workspace) return PATH_ERR_NULL;
    if ((log_f == nullptr) != (gc == nullptr)) return PATH_ERR_NULL;
    if (dt != PATH_BF16) return PATH_ERR_DTYPE;
    Plan p;
    if (cap < L || !make_plan(B, H, L, d, (int)dt, log_f ? 1 : 0, 0, p)) return PATH_ERR_SHAPE;
    if (!aligned16(k) || !aligned16(v) || !aligned16(w) || !aligned16(beta) || !aligned16(kc) || !aligned16(vc) ||
        (log_f && (!aligned16(log_f) || !aligned16(gc))) || ((uintptr_t)workspace & 255))
        return PATH_ERR_ALIGN;
    if (workspace_bytes < p.total) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, 256, st));
    // the chunk preparation needs no queries for the key side: the keys stand in for them
    const void* qd = k; const void* kd = k; const void* vd = v; const void* wd = w;
    rc = stage_inputs(p, workspace, qd, kd, vd, wd, beta, log_f, true, st);
    if (rc != PATH_OK) return rc;
    rc = run_prep(p, workspace, qd, kd, wd, false, st, false, true);
    if (rc != PATH_OK) return rc;
    LevelTensorMaps tm;
    if (!make_level_maps(p, workspace, tm)) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
    LevelParams lp = level_params(p, workspace);
    lp.cap = cap; lp.L = L;
    // A long prompt is cut into up to eight ranges of at least eight chunks per head: the serial walk over the chunks runs
    // per range (keys advanced to the range's end, bf16, in the unused plane of query tiles), then the ranges' products
    // are multiplied up towards the end of the sequence and applied, tile by tile, into the float32 cache.  The scratch
    // for the products is the (here unused) buffer of diagonal-correction operands.
    const int nseg = p.N >= 32 ? (p.N / 8 < 8 ? p.N / 8 : 8) : 1;
    if (nseg <= 1) {
        lp.kc = kc;
        LAUNCH(launch_level_kernel(LEVEL_KEY_CACHE, tm, lp, d, st));
    } else {
        typedef __nv_bfloat16 bf;
        const size_t mats = (size_t)p.S * nseg * 2 * d * d;          // elements of one [S][nseg][2][d][d] buffer
        bf* edge = at<bf>(workspace, p.Qv16);
        bf* pseg = at<bf>(workspace, p.Xqn);
        bf* sfx = pseg + mats;
        lp.nseg = nseg; lp.seg_chunks = (p.N + nseg - 1) / nseg;
        lp.edge16 = edge; lp.pseg = pseg; lp.sfx = sfx; lp.L = p.Lp;   // (whole padded chunks: padded rows are zero)
        LAUNCH(launch_level_kernel(LEVEL_KEY_CACHE, tm, lp, d, st));
        LevelTensorMaps tm2 = tm;
        if (!make_map(&tm2.dyh, pseg, (uint64_t)p.S * nseg * 2 * d, d)) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
        LAUNCH(launch_level_kernel(LEVEL_SUFFIX, tm2, lp, d, st));
        if (!(make_map(&tm2.dyh, sfx, (uint64_t)p.S * nseg * 2 * d, d) && make_map(&tm2.qv, edge, (uint64_t)p.S * p.Lp, d))) {
            g_last_cuda_error = (int)cudaErrorUnknown;
            return PATH_ERR_LAUNCH;
        }
        lp.kc = kc; lp.L = L; lp.edge16 = nullptr; lp.qv = edge; lp.gq = nullptr;
        LAUNCH(launch_level_kernel(LEVEL_APPLY_PRODUCT, tm2, lp, d, st));
    }
    CK(cudaMemcpy2DAsync(vc, (size_t)cap * d * 2, v, (size_t)L * d * 2, (size_t)L * d * 2, (size_t)p.S, cudaMemcpyDeviceToDevice, st));
    if (gc)
        CK(cudaMemcpy2DAsync(gc, (size_t)cap * 4, at<float>(workspace, p.G), (size_t)p.Lp * 4, (size_t)L * 4, (size_t)p.S,
                             cudaMemcpyDeviceToDevice, st));
    return PATH_OK;
}

size_t path_attn_decode_workspace_bytes(int B, int H, int cap, int d) {
    if (B < 1 || H < 1 || cap < 1 || (d != 64 && d != 128) || (long long)B * H > (1 << 20)) return 0;
    return 256 + ((decode_partials_bytes(B * H, cap, d) + 255) & ~(size_t)255);
}

int path_attn_decode_step(const void* q_t, const void* k_t, const void* v_t, const void* w_t, const float* beta_t,
                          const float* log_f_t, float* kc, void* vc, float* gc, int t, int cap, void* o_t, float* lse_t,
                          int B, int H, int d, float scale, path_dtype_t dt, void* workspace, size_t workspace_bytes,
                          void* cuda_stream) {
    g_launches = 0;
    if (!q_t || !k_t || !v_t || !w_t || !beta_t || !kc || !vc || !o_t || !lse_t || !workspace) return PATH_ERR_NULL;
    if ((log_f_t == nullptr) != (gc == nullptr)) return PATH_ERR_NULL;
    if (dt != PATH_BF16) return PATH_ERR_DTYPE;
    const size_t need = path_attn_decode_workspace_bytes(B, H, cap, d);
    if (need == 0 || t < 0 || t >= cap) return PATH_ERR_SHAPE;
    const void* ptrs[] = {q_t, k_t, v_t, w_t, kc, vc, o_t};
    for (const void* x : ptrs)
        if (!aligned16(x)) return PATH_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return PATH_ERR_ALIGN;
    if (workspace_bytes < need) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    LAUNCH(launch_decode_step(q_t, k_t, v_t, w_t, beta_t, log_f_t, kc, vc, gc, t, cap, o_t, lse_t, B * H, d, scale,
                              (float*)((uint8_t*)workspace + 256), st));
    return PATH_OK;
}

// ------------------------------------------------------------------------------------------- low-rank linear layer
// C[Mo, No] (+)= op(A) op(B) with a contraction of K; an operand given as [K][rows] enters transposed (MN-major).
static int run_gemm(const void* a, int a_mn, const void* b, int b_mn, void* c, int c_atomic, int Mo, int No, int K,
                    uint32_t* status, cudaStream_t st) {
    CUtensorMap ma, mb;
    const bool ok = (a_mn ? make_map_box(&ma, a, (uint64_t)K, (uint64_t)Mo, 64) : make_map_box(&ma, a, (uint64_t)Mo, (uint64_t)K, 128)) &&
                    (b_mn ? make_map_box(&mb, b, (uint64_t)K, (uint64_t)No, 64) : make_map_box(&mb, b, (uint64_t)No, (uint64_t)K, 128));
    if (!ok) { g_last_cuda_error = (int)cudaErrorUnknown; return PATH_ERR_LAUNCH; }
    GemmParams gp{};
    gp.M = Mo; gp.N = No; gp.K = K; gp.a_mn = a_mn; gp.b_mn = b_mn; gp.c = c; gp.ldc = No; gp.c_atomic = c_atomic; gp.status = status;
    int split = 1;
    if (c_atomic) {   // weight gradients: few output tiles, a contraction over all tokens: spread it over about two waves of CTAs
        const int tiles = ((Mo + 127) / 128) * ((No + 127) / 128), stages = (K + 63) / 64;
        split = 296 / tiles;
        split = split < 1 ? 1 : (split > stages ? stages : split);
    }
    LAUNCH(launch_gemm(ma, mb, gp, split, st));
    return PATH_OK;
}

static bool lowrank_shape_ok(long long M, int D, int r, int C) {
    return M >= 1 && M <= (1LL << 30) && D >= 64 && D % 64 == 0 && D <= (1 << 20) && (r == 64 || r == 128) && C >= 64 &&
           C % 64 == 0 && C <= (1 << 20);
}

size_t path_attn_lowrank_workspace_bytes(long long M, int D, int r, int C) {
    if (!lowrank_shape_ok(M, D, r, C)) return 0;
    return 256 + (((size_t)M * r * 2 + 255) & ~(size_t)255);
}

int path_attn_lowrank_fwd(const void* x, const void* w1, const void* w2, void* t, void* z, long long M, int D, int r, int C,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    g_launches = 0;
    if (!x || !w1 || !w2 || !t || !z || !workspace) return PATH_ERR_NULL;
    if (!lowrank_shape_ok(M, D, r, C)) return PATH_ERR_SHAPE;
    const void* ptrs[] = {x, w1, w2, t, z};
    for (const void* q_ : ptrs)
        if (!aligned16(q_)) return PATH_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return PATH_ERR_ALIGN;
    if (workspace_bytes < 256) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(workspace, 0, 256, st));
    rc = run_gemm(x, 0, w1, 0, t, 0, (int)M, r, D, (uint32_t*)workspace, st);         // t = x W1^T
    if (rc != PATH_OK) return rc;
    return run_gemm(t, 0, w2, 0, z, 0, (int)M, C, r, (uint32_t*)workspace, st);       // z = t W2^T
}

int path_attn_lowrank_bwd(const void* x, const void* w1, const void* w2, const void* t, const void* dz, void* dx, float* dw1,
                          float* dw2, long long M, int D, int r, int C, void* workspace, size_t workspace_bytes,
                          void* cuda_stream) {
    g_launches = 0;
    if (!x || !w1 || !w2 || !t || !dz || !dx || !dw1 || !dw2 || !workspace) return PATH_ERR_NULL;
    if (!lowrank_shape_ok(M, D, r, C)) return PATH_ERR_SHAPE;
    const void* ptrs[] = {x, w1, w2, t, dz, dx, dw1, dw2};
    for (const void* q_ : ptrs)
        if (!aligned16(q_)) return PATH_ERR_ALIGN;
    if ((uintptr_t)workspace & 255) return PATH_ERR_ALIGN;
    if (workspace_bytes < path_attn_lowrank_workspace_bytes(M, D, r, C)) return PATH_ERR_WORKSPACE;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    uint32_t* status = (uint32_t*)workspace;
    void* dt = (uint8_t*)workspace + 256;
    CK(cudaMemsetAsync(workspace, 0, 256, st));
    CK(cudaMemsetAsync(dw1, 0, (size_t)r * D * sizeof(float), st));
    CK(cudaMemsetAsync(dw2, 0, (size_t)C * r * sizeof(float), st));
    rc = run_gemm(dz, 0, w2, 1, dt, 0, (int)M, r, C, status, st);                     // dt = dz W2
    if (rc != PATH_OK) return rc;
    rc = run_gemm(dz, 1, t, 1, dw2, 1, C, r, (int)M, status, st);                     // dW2 = dz^T t
    if (rc != PATH_OK) return rc;
    rc = run_gemm(dt, 0, w1, 1, dx, 0, (int)M, D, r, status, st);                     // dx = dt W1
    if (rc != PATH_OK) return rc;
    return run_gemm(dt, 1, x, 1, dw1, 1, r, D, (int)M, status, st);                   // dW1 = dt^T x
}

// ------------------------------------------------------------------------------------------- layer front-end
static int frontend_shape_ok(int B, int H, int L, int d) {
    if (B < 1 || H < 1 || L < 1 || (d != 64 && d != 128)) return 0;
    const size_t blocks = ((size_t)L + 127) / 128 * (size_t)B * H;
    return blocks <= 0x7fffffffull;
}

int path_attn_frontend_fwd(const void* z, const float* conv_w, const float* beta_logit, const float* gate_logit, void* w,
                           float* beta, float* log_f, int B, int H, int L, int d, float eps, void* cuda_stream) {
    g_launches = 0;
    if (!z || !conv_w || !beta_logit || !w || !beta) return PATH_ERR_NULL;
    if ((gate_logit == nullptr) != (log_f == nullptr)) return PATH_ERR_NULL;
    if (!frontend_shape_ok(B, H, L, d) || !(eps >= 0.f)) return PATH_ERR_SHAPE;
    if (!aligned16(z) || !aligned16(w)) return PATH_ERR_ALIGN;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    LAUNCH(launch_frontend_fwd(z, conv_w, beta_logit, gate_logit, w, beta, log_f, B, H, L, d, eps, (cudaStream_t)cuda_stream));
    return PATH_OK;
}

int path_attn_frontend_bwd(const void* z, const float* conv_w, const float* beta_logit, const float* gate_logit, const void* dw,
                           const float* dbeta, const float* dlog_f, void* dz, float* dconv_w, float* dbeta_logit,
                           float* dgate_logit, int B, int H, int L, int d, float eps, void* cuda_stream) {
    g_launches = 0;
    if (!z || !conv_w || !beta_logit || !dw || !dbeta || !dz || !dconv_w || !dbeta_logit) return PATH_ERR_NULL;
    if ((gate_logit == nullptr) != (dlog_f == nullptr) || (gate_logit == nullptr) != (dgate_logit == nullptr)) return PATH_ERR_NULL;
    if (!frontend_shape_ok(B, H, L, d) || !(eps >= 0.f)) return PATH_ERR_SHAPE;
    if (!aligned16(z) || !aligned16(dw) || !aligned16(dz)) return PATH_ERR_ALIGN;
    int rc = check_arch();
    if (rc != PATH_OK) return rc;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CK(cudaMemsetAsync(dconv_w, 0, (size_t)H * d * 3 * sizeof(float), st));
    LAUNCH(launch_frontend_bwd(z, conv_w, beta_logit, gate_logit, dw, dbeta, dlog_f, dz, dconv_w, dbeta_logit, dgate_logit, B, H,
                               L, d, eps, st));
    return PATH_OK;
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
    return word == 0 ? PATH_OK : (word == ST_STATE ? PATH_ERR_STATE : PATH_ERR_TIMEOUT);
}

int path_attn_skipped_chunk_pairs(const void* workspace, void* cuda_stream, unsigned long long* kept,
                                  unsigned long long* all) {
    if (!workspace || !kept || !all) return PATH_ERR_NULL;
    unsigned long long c[2] = {0, 0};
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(c, (const uint8_t*)workspace + kSkipCounterOffset, sizeof(c), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        g_last_cuda_error = (int)cudaGetLastError();
        return PATH_ERR_LAUNCH;
    }
    *kept = c[0]; *all = c[1];
    return PATH_OK;
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
        case PATH_ERR_STATIC_LIMIT: return "problem needs more scratch than the built-in static buffer holds";
        case PATH_ERR_STATE: return "the workspace does not hold the forward state of this problem (path_attn_bwd_reuse)";
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
