// float32 GEMM for the float32 model (the tiny configuration): Y[m][n] = sum_k X[m][k] W[n][k].
// One warp per (output feature, group of 8 token rows); lanes stride over k and reduce by shuffles.
// Same output contract as the tensor-core kernel with a single split.
#include "kernels.h"

namespace tasc {

namespace {

constexpr int ROWS = 8;

__global__ void __launch_bounds__(128)
gemm_f32_kernel(const float* __restrict__ X, const float* __restrict__ W, float* __restrict__ P, int M, int N, int K,
                unsigned long long* argmax, float* logits) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n = blockIdx.x * 4 + warp;
    const int m0 = blockIdx.y * ROWS;
    if (n >= N) return;
    float acc[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) acc[r] = 0.f;
    const float* w = W + (size_t)n * K;
    for (int k = lane; k < K; k += 32) {
        const float wv = w[k];
#pragma unroll
        for (int r = 0; r < ROWS; ++r)
            if (m0 + r < M) acc[r] = fmaf(X[(size_t)(m0 + r) * K + k], wv, acc[r]);
    }
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        const float v = warp_sum(acc[r]);
        if (lane == 0 && m0 + r < M) {
            if (argmax) {
                atomicMax(&argmax[m0 + r], pack_argmax(v, (uint32_t)n));
                if (logits) logits[(size_t)(m0 + r) * N + n] = v;
            } else {
                P[(size_t)(m0 + r) * N + n] = v;
            }
        }
    }
}

}  // namespace

void launch_gemm_f32(const float* X, const float* W, float* partials, int M, int N, int K,
                     unsigned long long* argmax, float* logits, cudaStream_t stream) {
    ProfScope ps(argmax ? K_GEMM_LM : K_GEMM, stream);
    dim3 grid((N + 3) / 4, (M + ROWS - 1) / ROWS);
    gemm_f32_kernel<<<grid, 128, 0, stream>>>(X, W, partials, M, N, K, argmax, logits);
}

}  // namespace tasc
