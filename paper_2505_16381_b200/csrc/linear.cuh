// Batched small-matrix machinery of the chunk-level ("linear in L") part of PaTH attention:
// a generic tensor-core GEMM with masks / fused epilogues / batch addressing policies, the
// triangular inverse of the UT transform, padding, the gate prefix sum and small reductions.
#pragma once
#include "common.cuh"

namespace path {

// A(mn, k) = p[mn * s_mn + k * s_k], element type bf16 (f32 = 0) or float (f32 = 1).
struct Operand {
    const void* p;
    long s_mn, s_k;
    int f32;
};

enum { MASK_NONE = 0, MASK_LOWER = 1, MASK_STRICT = 2 };
enum { ACC_NONE = 0, ACC_ADD = 1, ACC_ATOMIC = 2 };

// C[m][n] = mask( alpha * sum_k A(m,k) B(k,n) + gamma * D[m][n] + identity ) (+ C_old)
// C2 (bf16, optional) = alpha2 * C, written as C2[m][n] or, if c2_trans, C2[n][m]; rows m >= c2_rows skipped.
struct GemmProblem {
    Operand A, B;
    int M, N, K;
    void* C; int c_f32; long ldc;
    void* C2; long ldc2; int c2_trans; float alpha2; int c2_rows;
    const void* D; int d_f32; long ldd; float gamma;
    float alpha;
    int accumulate, mask, identity;
    int split;  // float operands are split into two bf16 terms (three products) instead of rounded once
};

inline GemmProblem gemm_problem(Operand A, Operand B, int M, int N, int K) {
    GemmProblem g{};
    g.A = A; g.B = B; g.M = M; g.N = N; g.K = K;
    g.alpha = 1.f; g.alpha2 = 1.f; g.gamma = 1.f; g.c2_rows = 1 << 30; g.split = 1;
    return g;
}

// Two-level affine batch addressing: z -> (z0, z1) = (z / nb1, z % nb1); every pointer advances by
// z0 * s0 + z1 * s1 elements.  For C2 the valid row count is min(128, rows_total - z1 * 128) when
// rows_total > 0 (ragged tail of the user's [S, L, d] tensors).
struct AffineBatch {
    int nb1;
    long a0, a1, b0, b1, c0, c1, c20, c21, d0, d1;
    int rows_total;
};

struct LevelTable {
    long dy_off[20];   // element offset of level l inside the Dy buffer
    int dy_cnt[20];    // runs per slice at level l  (N >> l)
};

// Version chains (see common.cuh for the slot convention).  mode 0: forward  Xv[l2] = Xv[l1] * Dy (queries) or
// Dy^T (keys).  mode 1: backward data  dXv[l1] += dXv[l2] * Dy^T (queries) or Dy (keys).  mode 2: backward
// product  dDy[l1][b] += Xv[l1]^T dXv[l2] (queries) or dXv[l2]^T Xv[l1] (keys), atomically.
struct VersionBatch {
    int is_key, mode, l2, S, N, Lp, d;
    LevelTable lv;
    const __nv_bfloat16* xv;  // [slots][S][Lp][d] bf16 versions (what the attention kernels consume)
    float* dxv;               // float gradients, same layout (modes 1, 2)
    const float* dy;          // dyadic run products
    float* ddy;               // their gradients (mode 2)
    __nv_bfloat16* out16;     // mode 0: destination (same buffer as xv)
};

cudaError_t launch_gemm(const GemmProblem& g, const AffineBatch& b, int nbatch, cudaStream_t st);
cudaError_t launch_gemm_version(const VersionBatch& v, cudaStream_t st);

// Ainv = (I + strictLower(diag(beta) Gm))^-1 and Tt = Ainv diag(beta), per 128 x 128 chunk.
cudaError_t launch_tri_inverse(const float* Gm, const float* beta, float* Ainv, float* Tt, int nchunks,
                               cudaStream_t st);
// dst[S][Lp][d] <- src[S][L][d] (zero tail); bf16 elements when !f32.
cudaError_t launch_pad_rows(const void* src, void* dst, int S, int L, int Lp, int d, int f32, cudaStream_t st);
// dst[S][Lp] <- src[S][L] (zero tail), float.
cudaError_t launch_pad_vec(const float* src, float* dst, int S, int L, int Lp, cudaStream_t st);
// G[S][Lp] <- inclusive prefix sum of g[S][L] (tail repeats the last value).
cudaError_t launch_gate_prefix(const float* g, float* G, int S, int L, int Lp, cudaStream_t st);

// Pieces of the UT-transform chain rule that are not matrix products (see path_attn.cu, chunk chain rule).
cudaError_t launch_beta_cols(const float* Ainv, float* dT, const float* beta, float* t1, int nchunks, cudaStream_t st);
cudaError_t launch_beta_rows(float* dA, const float* Gm, const float* beta, const float* t1, float* dbeta, int S, int N,
                             int L, cudaStream_t st);
// out[S][L] <- reverse inclusive prefix sum of (dGa + dGb + dGc)[S][Lp] over positions < L.
cudaError_t launch_gate_suffix(const float* dGa, const float* dGb, const float* dGc, float* out, int S, int L, int Lp,
                               cudaStream_t st);
// rs[chunk][i] = sum_k dsd[chunk][i][k]
cudaError_t launch_dsd_rowsum(const float* dsd, float* rs, int nchunks, cudaStream_t st);

}  // namespace path
