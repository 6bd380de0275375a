// Small memory-bound helpers around the tile kernels: padding of ragged inputs, the gate's prefix and suffix
// sums and a row reduction.
#pragma once
#include "common.cuh"

namespace path {

// dst[S][Lp][d] <- src[S][L][d] (zero tail); bf16 elements when !f32.
cudaError_t launch_pad_rows(const void* src, void* dst, int S, int L, int Lp, int d, int f32, cudaStream_t st);
// dst[S][Lp] <- src[S][L] (zero tail), float.
cudaError_t launch_pad_vec(const float* src, float* dst, int S, int L, int Lp, cudaStream_t st);
// G[S][Lp] <- inclusive prefix sum of g[S][L] (tail repeats the last value).
cudaError_t launch_gate_prefix(const float* g, float* G, int S, int L, int Lp, cudaStream_t st);

// out[S][L] <- reverse inclusive prefix sum of (dGa + dGb + dGc)[S][Lp] over positions < L.
cudaError_t launch_gate_suffix(const float* dGa, const float* dGb, const float* dGc, float* out, int S, int L, int Lp,
                               cudaStream_t st);
// rs[chunk][i] = sum_k dsd[chunk][i][k]
cudaError_t launch_dsd_rowsum(const float* dsd, float* rs, int nchunks, cudaStream_t st);

// Gated problems (PaTH-FoX): which key chunks a query chunk can skip because the accumulated gate has made every logit
// of the pair negligible.  stats: [S*N][8] floats of scratch; nkeep: [S*N] key chunks each query chunk visits (counted
// from the diagonal); nvisit: [S*N] query chunks each key chunk meets (the same pairs, key-major); counters: {kept pairs,
// all pairs}, added to (zeroed by the caller).  q, k, w: [S][Lp][hd] bf16 (padded), beta, G: [S][Lp].
cudaError_t launch_gate_skip(const void* q, const void* k, const void* w, const float* beta, const float* G, float* stats,
                             int* nkeep, int* nvisit, unsigned long long* counters, int S, int L, int Lp, int hd, float scale,
                             cudaStream_t st);

// Context-parallel path (paper Sec. 3.5), gate terms of a segment from its prefix sums G [S][Lp] (nullptr = no gate):
// gq[S][Lp] <- G (the query rows' terms), gk[S][Lp] <- G - G[L-1] for positions < L and a huge value for the padded tail
// (which masks those keys), gtot[S] <- G[L-1].
cudaError_t launch_cp_gate(const float* G, float* gq, float* gk, float* gtot, int S, int L, int Lp, cudaStream_t st);
// Running softmax state (o_acc [S][L][d] float32 normalised, lse_acc [S][L]) merged with a partial result of the same
// shape (o_t, lse_t): o_acc <- (e^{lse_acc} o_acc + e^{lse_t} o_t) / (e^{lse_acc} + e^{lse_t}), lse_acc <- log of that sum.
cudaError_t launch_cp_merge(float* o_acc, float* lse_acc, const float* o_t, const float* lse_t, size_t rows, int hd,
                            cudaStream_t st);
// o [rows][d] bf16 <- o_acc, lse <- lse_acc.
cudaError_t launch_cp_finish(const float* o_acc, const float* lse_acc, void* o, float* lse, size_t rows, int hd,
                             cudaStream_t st);

// Forward-state record in the status block of a workspace (see StateRecord): written at the end of a forward that kept its
// chunk preparation, compared by the backward that wants to reuse it (a mismatch raises ST_STATE in the status word).
cudaError_t launch_state_write(void* record, const StateRecord& rec, cudaStream_t st);
cudaError_t launch_state_check(const void* record, const StateRecord& want, uint32_t* status, cudaStream_t st);
// One thread waits on an mbarrier that nothing arrives on, with a limit of `ticks` clock cycles, then reports
// ST_SELFTEST through the status word like every bounded wait of the library does.
cudaError_t launch_selftest_wait(uint32_t* status, long long ticks, cudaStream_t st);

}  // namespace path
