// Dense refit for sequential compression (appendix "Sequential Quantization with OBQ" of "Optimal Brain
// Compression"): when a layer's inputs X are those of the already compressed model, the dense weights are first
// re-optimised in closed form, W^T = (X X^T)^-1 X Y^T with Y the dense model's outputs, so that they are a
// minimiser again before the layer is compressed.  Two steps, both accumulating like the Hessian:
//     G (+)= Y X^T                       (tensor cores for TF32 / BF16X3, CUDA cores for FP32)
//     W  = 2 G Hinv,  Hinv = inv(2 X X^T + lambda I)   (the dampened inverse the solver uses anyway)
// This file holds the FP32 CUDA-core product C = alpha A B^T used by both steps.
#include "common.cuh"

namespace obc {

constexpr int RT = 64;            // output tile
constexpr int RK = 16;            // k chunk

// C (M x N, ldc) = alpha * A (M x K, lda) * B^T (B is N x K, ldb) + beta * C; row-major FP32.
__global__ void __launch_bounds__(256) sgemm_nt_kernel(int M, int N, int64_t K, float alpha, const float* __restrict__ A,
                                                       int64_t lda, const float* __restrict__ B, int64_t ldb, float beta,
                                                       float* __restrict__ C, int ldc) {
    __shared__ float As[RK][RT + 1];
    __shared__ float Bs[RK][RT + 1];
    const int bm = blockIdx.y * RT, bn = blockIdx.x * RT;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    float acc[4][4] = {};
    for (int64_t k0 = 0; k0 < K; k0 += RK) {
        for (int e = tid; e < RT * RK; e += 256) {
            const int k = e % RK, i = e / RK;
            const int64_t gk = k0 + k;
            As[k][i] = (bm + i < M && gk < K) ? A[(size_t)(bm + i) * lda + gk] : 0.f;
            Bs[k][i] = (bn + i < N && gk < K) ? B[(size_t)(bn + i) * ldb + gk] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < RK; ++k) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[k][ty + 16 * i]; b[i] = Bs[k][tx + 16 * i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gi = bm + ty + 16 * i, gj = bn + tx + 16 * j;
            if (gi < M && gj < N) {
                float* c = C + (size_t)gi * ldc + gj;
                *c = (beta == 0.f ? 0.f : beta * *c) + alpha * acc[i][j];
            }
        }
}

obc_status sgemm_nt_launch(int M, int N, int64_t K, float alpha, const float* A, int64_t lda, const float* B, int64_t ldb,
                           float beta, float* C, int ldc, cudaStream_t stream) {
    dim3 grid((N + RT - 1) / RT, (M + RT - 1) / RT);
    sgemm_nt_kernel<<<grid, 256, 0, stream>>>(M, N, K, alpha, A, lda, B, ldb, beta, C, ldc);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

}  // namespace obc
