// Dampened inverse of the layer Hessian (Section 3, "Implementation Details" of "Optimal Brain
// Compression"): Hinv = inv(H + damp_rel * mean(diag H) * I).
//
// One d^3 job per layer, carried in FP64 so that the FP32 result is correctly rounded to well below the
// elimination engine's own error:  A = H + lambda I  ->  blocked right-looking Cholesky A = L L^T
// (48-wide panels; diagonal block factored and inverted by one CTA, panel solved against the inverted
// diagonal block, trailing matrix updated by a tiled FP64 GEMM)  ->  inverse of L by block doubling  ->
// Hinv = L^-T L^-1 (lower tiles) -> mirrored, exactly symmetric FP32 output.
#include "common.cuh"

namespace obc {

constexpr int NB = 48;            // panel width (two NB x NB FP64 blocks fit static shared memory)
constexpr int GT = 64;            // GEMM tile
constexpr int GK = 16;

// C (MxN) = beta*C + alpha * op(A) (MxK) * op(B) (KxN); row-major doubles.  TA: A is stored KxM.  TB: B is
// stored NxK.  lower_only: skip tiles strictly above the diagonal (M == N outputs that are symmetric).
// k_lo_from_tile: the product only needs k >= max(first row, first column) of the tile (L^-T L^-1).
template <bool TA, bool TB>
__device__ __forceinline__ void dgemm_tile(int M, int N, double alpha, const double* __restrict__ A, int lda,
                                           const double* __restrict__ B, int ldb, double beta, double* __restrict__ C,
                                           int ldc, int bm, int bn, int k_begin, int k_end) {
    __shared__ double As[GK][GT + 1];
    __shared__ double Bs[GK][GT + 1];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    double acc[4][4] = {};
    for (int k0 = k_begin; k0 < k_end; k0 += GK) {
        for (int e = tid; e < GT * GK; e += 256) {
            int i, k;
            if (TA) { i = e % GT; k = e / GT; } else { k = e % GK; i = e / GK; }
            const int gi = bm + i, gk = k0 + k;
            double v = 0.0;
            if (gi < M && gk < k_end) v = TA ? A[(size_t)gk * lda + gi] : A[(size_t)gi * lda + gk];
            As[k][i] = v;
        }
        for (int e = tid; e < GT * GK; e += 256) {
            int j, k;
            if (TB) { k = e % GK; j = e / GK; } else { j = e % GT; k = e / GT; }
            const int gj = bn + j, gk = k0 + k;
            double v = 0.0;
            if (gj < N && gk < k_end) v = TB ? B[(size_t)gj * ldb + gk] : B[(size_t)gk * ldb + gj];
            Bs[k][j] = v;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < GK; ++k) {
            double a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[k][ty + 16 * i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gi = bm + ty + 16 * i, gj = bn + tx + 16 * j;
            if (gi < M && gj < N) {
                double* c = C + (size_t)gi * ldc + gj;
                *c = (beta == 0.0 ? 0.0 : beta * *c) + alpha * acc[i][j];
            }
        }
}

template <bool TA, bool TB>
__global__ void __launch_bounds__(256) dgemm_kernel(int M, int N, int K, double alpha, const double* __restrict__ A, int lda,
                                                    const double* __restrict__ B, int ldb, double beta,
                                                    double* __restrict__ C, int ldc, int lower_only, int k_lo_from_tile) {
    const int bm = blockIdx.y * GT, bn = blockIdx.x * GT;
    if (lower_only && bn > bm + GT - 1) return;
    int k0 = 0;
    if (k_lo_from_tile) k0 = (max(bm, bn) / GK) * GK;
    dgemm_tile<TA, TB>(M, N, alpha, A, lda, B, ldb, beta, C, ldc, bm, bn, k0, K);
}

// One level of the recursive inverse of the lower-triangular factor.  With the inverses of the diagonal blocks of
// size s known, the diagonal blocks of size 2s follow from
//      inv([[L11, 0], [L21, L22]]) = [[X11, 0], [-X22 L21 X11, X22]] ,   X11 = inv(L11), X22 = inv(L22),
// for all pairs of blocks at once (blockIdx.z = pair; the last pair may be short or lack its second block).
// stage 0:  T = L21 * X11  (into the scratch matrix at the position of L21);  stage 1:  X21 = -X22 * T.
// X11 and X22 are lower triangular, which bounds the k range of every tile.
__global__ void __launch_bounds__(256) trinv_level_kernel(const double* __restrict__ L, double* __restrict__ X,
                                                          double* __restrict__ T, int d, int s, int stage) {
    const int lo = blockIdx.z * 2 * s;
    const int s1 = min(s, d - lo);
    const int s2 = min(s, d - lo - s);
    if (s2 <= 0) return;
    const int bm = blockIdx.y * GT, bn = blockIdx.x * GT;
    if (bm >= s2 || bn >= s1) return;
    const size_t o21 = (size_t)(lo + s) * d + lo, o11 = (size_t)lo * d + lo, o22 = (size_t)(lo + s) * d + lo + s;
    if (stage == 0)      // (T)[i][j] = sum_{k >= j} L21[i][k] X11[k][j]
        dgemm_tile<false, false>(s2, s1, 1.0, L + o21, d, X + o11, d, 0.0, T + o21, d, bm, bn, (bn / GK) * GK, s1);
    else                 // X21[i][j] = -sum_{k <= i} X22[i][k] T[k][j]
        dgemm_tile<false, false>(s2, s1, -1.0, X + o22, d, T + o21, d, 0.0, X + o21, d, bm, bn, 0, min(s2, bm + GT));
}

template <bool TA, bool TB>
static void dgemm(cudaStream_t s, int M, int N, int K, double alpha, const double* A, int lda, const double* B, int ldb,
                  double beta, double* C, int ldc, int lower_only = 0, int k_lo = 0) {
    if (M <= 0 || N <= 0) return;
    dim3 grid((N + GT - 1) / GT, (M + GT - 1) / GT);
    dgemm_kernel<TA, TB><<<grid, 256, 0, s>>>(M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, lower_only, k_lo);
    count_launch();
}

// trace of H (FP32) -> lambda; single block
__global__ void __launch_bounds__(256) damp_kernel(const float* __restrict__ H, int ldh, int d, float damp_rel,
                                                   double* __restrict__ lambda, int32_t* info) {
    __shared__ double part[256];
    double s = 0.0;
    for (int i = threadIdx.x; i < d; i += 256) s += (double)H[(size_t)i * ldh + i];
    part[threadIdx.x] = s;
    __syncthreads();
    for (int off = 128; off; off >>= 1) {
        if (threadIdx.x < off) part[threadIdx.x] += part[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) { *lambda = (double)damp_rel * part[0] / (double)d; *info = 0; }
}

// A = (double)H + lambda I  (lower triangle is what the factorisation reads);  Li = 0
__global__ void widen_kernel(const float* __restrict__ H, int ldh, int d, const double* __restrict__ lambda,
                             double* __restrict__ A, double* __restrict__ Li) {
    const size_t n = (size_t)d * d;
    const double lam = *lambda;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / d), j = (int)(e % d);
        A[e] = (double)H[(size_t)i * ldh + j] + (i == j ? lam : 0.0);
        Li[e] = 0.0;
    }
}

// Factor the nb x nb diagonal block at k0 in place (lower Cholesky) and write its inverse into Li.
__global__ void __launch_bounds__(256) chol_diag_kernel(double* __restrict__ A, double* __restrict__ Li, int d, int k0,
                                                        int nb, int32_t* info) {
    __shared__ double L[NB][NB + 1];
    __shared__ double X[NB][NB + 1];
    __shared__ int bad;
    const int tid = threadIdx.x;
    if (tid == 0) bad = 0;
    for (int e = tid; e < nb * nb; e += 256) {
        const int i = e / nb, j = e % nb;
        L[i][j] = j <= i ? A[(size_t)(k0 + i) * d + k0 + j] : 0.0;
    }
    __syncthreads();
    for (int j = 0; j < nb; ++j) {
        if (tid == 0) {
            const double s = L[j][j];
            if (!(s > 0.0) || !isfinite(s)) { if (!bad) { bad = 1; atomicCAS(info, 0, 1 + k0 + j); } L[j][j] = 1.0; }
            else L[j][j] = sqrt(s);
        }
        __syncthreads();
        const double ljj = L[j][j];
        for (int i = j + 1 + tid; i < nb; i += 256) L[i][j] /= ljj;
        __syncthreads();
        // trailing update of the block: L[i][c] -= L[i][j] * L[c][j] for j < c <= i
        const int rem = nb - j - 1;
        for (int e = tid; e < rem * rem; e += 256) {
            const int i = j + 1 + e / rem, c = j + 1 + e % rem;
            if (c <= i) L[i][c] -= L[i][j] * L[c][j];
        }
        __syncthreads();
    }
    // X = inv(L): column c solved by thread c (forward substitution)
    if (tid < nb) {
        const int c = tid;
        for (int i = 0; i < nb; ++i) {
            if (i < c) { X[i][c] = 0.0; continue; }
            double t = (i == c) ? 1.0 : 0.0;
            for (int k = c; k < i; ++k) t -= L[i][k] * X[k][c];
            X[i][c] = t / L[i][i];
        }
    }
    __syncthreads();
    for (int e = tid; e < nb * nb; e += 256) {
        const int i = e / nb, j = e % nb;
        if (j <= i) A[(size_t)(k0 + i) * d + k0 + j] = L[i][j];
        Li[(size_t)(k0 + i) * d + k0 + j] = X[i][j];
    }
}

// Panel below the diagonal block: A21 <- A21 * inv(L11)^T, 64 rows per block, in place.
__global__ void __launch_bounds__(256) chol_panel_kernel(double* __restrict__ A, const double* __restrict__ Li, int d,
                                                         int k0, int nb) {
    __shared__ double R[GT][NB + 1];
    __shared__ double X[NB][NB + 1];
    const int tid = threadIdx.x;
    const int i0 = k0 + nb + blockIdx.x * GT;
    const int rows = min(GT, d - i0);
    for (int e = tid; e < nb * nb; e += 256) { const int i = e / nb, j = e % nb; X[i][j] = Li[(size_t)(k0 + i) * d + k0 + j]; }
    for (int e = tid; e < rows * nb; e += 256) { const int i = e / nb, j = e % nb; R[i][j] = A[(size_t)(i0 + i) * d + k0 + j]; }
    __syncthreads();
    for (int e = tid; e < rows * nb; e += 256) {
        const int i = e / nb, j = e % nb;
        double t = 0.0;
        for (int k = 0; k <= j; ++k) t += R[i][k] * X[j][k];
        A[(size_t)(i0 + i) * d + k0 + j] = t;
    }
}

// Hinv32[i][j] = Hinv32[j][i] = (float) C[max(i,j)][min(i,j)]
__global__ void narrow_kernel(const double* __restrict__ C, int d, float* __restrict__ Hinv, int ldhi) {
    const size_t n = (size_t)d * d;
    for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / d), j = (int)(e % d);
        const int a = i > j ? i : j, b = i > j ? j : i;
        Hinv[(size_t)i * ldhi + j] = (float)C[(size_t)a * d + b];
    }
}

size_t inverse_workspace_bytes(int d) {
    const size_t mat = round_up((size_t)d * d * sizeof(double), 256);
    return 3 * mat + round_up((size_t)NB * d * sizeof(double), 256) + 256;
}

obc_status inverse_launch(const float* H, int d, int ldh, float damp_rel, float* Hinv, int ldhi, int32_t* info,
                          void* ws, cudaStream_t s) {
    const size_t mat = round_up((size_t)d * d * sizeof(double), 256);
    char* p = reinterpret_cast<char*>(ws);
    double* A = reinterpret_cast<double*>(p); p += mat;
    double* Li = reinterpret_cast<double*>(p); p += mat;
    double* C = reinterpret_cast<double*>(p); p += mat;
    p += round_up((size_t)NB * d * sizeof(double), 256);         // (reserved)
    double* lambda = reinterpret_cast<double*>(p);

    damp_kernel<<<1, 256, 0, s>>>(H, ldh, d, damp_rel, lambda, info);
    count_launch();
    widen_kernel<<<592, 256, 0, s>>>(H, ldh, d, lambda, A, Li);
    count_launch();
    // blocked Cholesky, lower, in place
    for (int k0 = 0; k0 < d; k0 += NB) {
        const int nb = d - k0 < NB ? d - k0 : NB;
        chol_diag_kernel<<<1, 256, 0, s>>>(A, Li, d, k0, nb, info);
        count_launch();
        const int below = d - k0 - nb;
        if (below > 0) {
            chol_panel_kernel<<<(below + GT - 1) / GT, 256, 0, s>>>(A, Li, d, k0, nb);
            count_launch();
            const double* P = A + (size_t)(k0 + nb) * d + k0;
            dgemm<false, true>(s, below, below, nb, -1.0, P, d, P, d, 1.0, A + (size_t)(k0 + nb) * d + k0 + nb, d, 1, 0);
        }
    }
    // inverse of L by block doubling: the diagonal NB-blocks of Li are known from the factorisation; each level
    // fills the off-diagonal halves of the diagonal blocks of twice the size, all pairs in one launch (C = scratch)
    for (int bs = NB; bs < d; bs *= 2) {
        const int pairs = (d + 2 * bs - 1) / (2 * bs);
        dim3 grid((bs + GT - 1) / GT, (bs + GT - 1) / GT, pairs);
        trinv_level_kernel<<<grid, 256, 0, s>>>(A, Li, C, d, bs, 0);
        trinv_level_kernel<<<grid, 256, 0, s>>>(A, Li, C, d, bs, 1);
        count_launch(2);
    }
    // C = Li^T Li on the lower tiles, then mirror into FP32
    dgemm<true, false>(s, d, d, d, 1.0, Li, d, Li, d, 0.0, C, d, 1, 1);
    narrow_kernel<<<592, 256, 0, s>>>(C, d, Hinv, ldhi);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

}  // namespace obc
