// Memory-bound helpers: zero-padding of ragged inputs, prefix sum of the log gate (PaTH-FoX, paper Sec. 2.2),
// suffix sum of its gradient, row sums of the diagonal-chunk dS.
#include "linear.cuh"

namespace path {

namespace {

__global__ void pad_rows_kernel(const void* __restrict__ src, void* __restrict__ dst, int L, int Lp, int rowbytes16) {
    // one 16-byte vector per thread; grid.y = slice, grid.x covers Lp * rowbytes16
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    const long total = (long)Lp * rowbytes16;
    if (i >= total) return;
    const long row = i / rowbytes16, col = i % rowbytes16;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < L) v = ((const uint4*)src)[((long)blockIdx.y * L + row) * rowbytes16 + col];
    ((uint4*)dst)[((long)blockIdx.y * Lp + row) * rowbytes16 + col] = v;
}

__global__ void pad_vec_kernel(const float* __restrict__ src, float* __restrict__ dst, int L, int Lp) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < Lp) dst[(size_t)blockIdx.y * Lp + i] = (i < L) ? src[(size_t)blockIdx.y * L + i] : 0.f;
}

// One CTA (1024 threads) per slice: each thread scans a contiguous segment, then a block scan of the segment sums.
__global__ void __launch_bounds__(1024) gate_prefix_kernel(const float* __restrict__ g, float* __restrict__ G, int L,
                                                           int Lp) {
    __shared__ float part[1024];
    const int tid = threadIdx.x;
    const int seg = (Lp + 1023) / 1024;
    const int lo = tid * seg, hi = min(lo + seg, Lp);
    const float* gs = g + (size_t)blockIdx.x * L;
    float* Gs = G + (size_t)blockIdx.x * Lp;
    float acc = 0.f;
    for (int i = lo; i < hi; ++i) acc += (i < L) ? gs[i] : 0.f;
    part[tid] = acc;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        float v = (tid >= off) ? part[tid - off] : 0.f;
        __syncthreads();
        part[tid] += v;
        __syncthreads();
    }
    acc = (tid > 0) ? part[tid - 1] : 0.f;
    for (int i = lo; i < hi; ++i) {
        acc += (i < L) ? gs[i] : 0.f;
        Gs[i] = acc;
    }
}

// rs[chunk*128 + i] = sum_k dsd[chunk][i][k]; one warp per row.
__global__ void __launch_bounds__(256) dsd_rowsum_kernel(const float* __restrict__ dsd, float* __restrict__ rs) {
    const size_t base = (size_t)blockIdx.x * CHUNK * CHUNK;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r < CHUNK; r += 8) {
        float acc = 0.f;
        for (int c = lane; c < CHUNK; c += 32) acc += dsd[base + r * CHUNK + c];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0) rs[(size_t)blockIdx.x * CHUNK + r] = acc;
    }
}

// dlog_f[t] = sum_{m >= t} (dGa + dGb + dGc)[m]: reverse inclusive scan per slice (inputs [S][Lp], output [S][L]).
__global__ void __launch_bounds__(1024) gate_suffix_kernel(const float* __restrict__ dGa, const float* __restrict__ dGb,
                                                           const float* __restrict__ dGc, float* __restrict__ out, int L,
                                                           int Lp) {
    __shared__ float part[1024];
    const int tid = threadIdx.x;
    const int seg = (L + 1023) / 1024;
    const int hi = L - tid * seg, lo = max(hi - seg, 0);  // this thread owns positions [lo, hi), scanning downwards
    const size_t so = (size_t)blockIdx.x * Lp;
    float* os = out + (size_t)blockIdx.x * L;
    float acc = 0.f;
    for (int i = hi - 1; i >= lo; --i) acc += (dGa[so + i] + dGb[so + i]) + dGc[so + i];
    part[tid] = acc;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {
        float v = (tid >= off) ? part[tid - off] : 0.f;
        __syncthreads();
        part[tid] += v;
        __syncthreads();
    }
    acc = (tid > 0) ? part[tid - 1] : 0.f;
    for (int i = hi - 1; i >= lo; --i) {
        acc += (dGa[so + i] + dGb[so + i]) + dGc[so + i];
        os[i] = acc;
    }
}

}  // namespace

cudaError_t launch_gate_suffix(const float* dGa, const float* dGb, const float* dGc, float* out, int S, int L, int Lp,
                               cudaStream_t st) {
    gate_suffix_kernel<<<S, 1024, 0, st>>>(dGa, dGb, dGc, out, L, Lp);
    return cudaGetLastError();
}
cudaError_t launch_dsd_rowsum(const float* dsd, float* rs, int nchunks, cudaStream_t st) {
    dsd_rowsum_kernel<<<nchunks, 256, 0, st>>>(dsd, rs);
    return cudaGetLastError();
}

cudaError_t launch_pad_rows(const void* src, void* dst, int S, int L, int Lp, int d, int f32, cudaStream_t st) {
    const int rowbytes16 = d * (f32 ? 4 : 2) / 16;
    const long total = (long)Lp * rowbytes16;
    dim3 grid((unsigned)((total + 255) / 256), S);
    pad_rows_kernel<<<grid, 256, 0, st>>>(src, dst, L, Lp, rowbytes16);
    return cudaGetLastError();
}

cudaError_t launch_pad_vec(const float* src, float* dst, int S, int L, int Lp, cudaStream_t st) {
    dim3 grid((Lp + 255) / 256, S);
    pad_vec_kernel<<<grid, 256, 0, st>>>(src, dst, L, Lp);
    return cudaGetLastError();
}

cudaError_t launch_gate_prefix(const float* g, float* G, int S, int L, int Lp, cudaStream_t st) {
    gate_prefix_kernel<<<S, 1024, 0, st>>>(g, G, L, Lp);
    return cudaGetLastError();
}

}  // namespace path
