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

}  // namespace path
