// C[M, N] = A[M, K] * W[N, K]^T with float accumulation on the plain FP32 pipes.
// Used for float32 models (TF32 tensor cores would break their 1e-4 logit tolerance) and as the
// reference the tensor-core GEMMs are checked against.  Each output element sums its K products in
// a fixed order that does not depend on M, so a row's result does not depend on its batch mates.
#pragma once

#include "common.cuh"

namespace pc {

// Epilogues receive four consecutive columns [col0, col0+4) of one row; n_valid of them are inside N.
struct EpiStoreF32 {            // C = acc (+ bias)
    float* C; int ldc; const float* bias;
    __device__ __forceinline__ void operator()(int row, int col0, const float* acc, int n_valid) const {
        for (int i = 0; i < n_valid; ++i)
            C[(size_t)row * ldc + col0 + i] = acc[i] + (bias ? bias[col0 + i] : 0.f);
    }
};
struct EpiResidual {            // H += acc   (float residual stream)
    float* H; int ldc;
    __device__ __forceinline__ void operator()(int row, int col0, const float* acc, int n_valid) const {
        for (int i = 0; i < n_valid; ++i) H[(size_t)row * ldc + col0 + i] += acc[i];
    }
};
template <typename T>
struct EpiSwiGLU {              // columns (2j, 2j+1) = (gate_j, up_j)  ->  out[row, j] = silu(gate) * up
    T* out; int ld;
    __device__ __forceinline__ void operator()(int row, int col0, const float* acc, int n_valid) const {
        for (int i = 0; i + 1 < n_valid; i += 2) {
            const float g = acc[i], u = acc[i + 1];
            out[(size_t)row * ld + ((col0 + i) >> 1)] = from_f32<T>(g / (1.f + expf(-g)) * u);
        }
    }
};

template <typename T, class Epi>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const StepDesc* __restrict__ sd, const T* __restrict__ A, const T* __restrict__ W, int M, int N, int K, Epi epi) {
    if (sd != nullptr) M = sd->n_rows;          // live row count; the grid was sized for an upper bound
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 4];
    __shared__ float Ws[BK][BN + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    if (m0 >= M) return;
    const int lrow = tid >> 2, lk = (tid & 3) * 4;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += BK) {
        float va[4] = {0.f, 0.f, 0.f, 0.f}, vw[4] = {0.f, 0.f, 0.f, 0.f};
        if (k0 + lk < K) {          // K is a multiple of 4
            if (m0 + lrow < M) VecLoad<T, 4>::load(A + (size_t)(m0 + lrow) * K + k0 + lk, va);
            if (n0 + lrow < N) VecLoad<T, 4>::load(W + (size_t)(n0 + lrow) * K + k0 + lk, vw);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) { As[lk + i][lrow] = va[i]; Ws[lk + i][lrow] = vw[i]; }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
    }
    const int col0 = n0 + tx * 4;
    if (col0 >= N) return;
    const int n_valid = min(4, N - col0);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = m0 + ty * 4 + i;
        if (row < M) epi(row, col0, acc[i], n_valid);
    }
}

template <typename T, class Epi>
inline void launch_gemm_simt(cudaStream_t st, const StepDesc* sd, const T* A, const T* W, int M, int N, int K, Epi epi) {
    if (M <= 0 || N <= 0) return;
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    gemm_simt_kernel<T, Epi><<<grid, 256, 0, st>>>(sd, A, W, M, N, K, epi);
}

}  // namespace pc
