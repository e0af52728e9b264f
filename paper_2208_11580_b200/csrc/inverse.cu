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
// C may be A itself when N <= GT and A is not transposed: a CTA then reads its own rows completely before it
// writes them, and no other CTA touches them.
// k_lo_from_tile: the product only needs k >= max(first row, first column) of the tile (L^-T L^-1).
template <bool TA, bool TB>
__device__ __forceinline__ void dgemm_tile(int M, int N, double alpha, const double* A, int lda,
                                           const double* __restrict__ B, int ldb, double beta, double* C,
                                           int ldc, int bm, int bn, int k_begin, int k_end) {
    __shared__ double As[GK][GT + 1];
    __shared__ double Bs[GK][GT + 1];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    double acc[4][4] = {};
    // element e = tid + 256 r of a GT x GK operand tile; the next chunk's elements are fetched into registers
    // while the current chunk is multiplied
    double ra[4], rb[4];
    auto fetch = [&](int k0) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int e = tid + 256 * r;
            int i, k;
            if (TA) { i = e % GT; k = e / GT; } else { k = e % GK; i = e / GK; }
            const int gi = bm + i, gk = k0 + k;
            ra[r] = (gi < M && gk < k_end) ? (TA ? A[(size_t)gk * lda + gi] : A[(size_t)gi * lda + gk]) : 0.0;
            int j, kb;
            if (TB) { kb = e % GK; j = e / GK; } else { j = e % GT; kb = e / GT; }
            const int gj = bn + j, gkb = k0 + kb;
            rb[r] = (gj < N && gkb < k_end) ? (TB ? B[(size_t)gj * ldb + gkb] : B[(size_t)gkb * ldb + gj]) : 0.0;
        }
    };
    if (k_begin < k_end) fetch(k_begin);
    for (int k0 = k_begin; k0 < k_end; k0 += GK) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int e = tid + 256 * r;
            if (TA) As[e / GT][e % GT] = ra[r]; else As[e % GK][e / GK] = ra[r];
            if (TB) Bs[e % GK][e / GK] = rb[r]; else Bs[e / GT][e % GT] = rb[r];
        }
        __syncthreads();
        if (k0 + GK < k_end) fetch(k0 + GK);
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
__global__ void __launch_bounds__(256) dgemm_kernel(int M, int N, int K, double alpha, const double* A, int lda,
                                                    const double* __restrict__ B, int ldb, double beta,
                                                    double* C, int ldc, int lower_only, int k_lo_from_tile) {
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
// 16 x 16 threads, each holding a 3 x 3 sub-grid (rows ty + 16p, columns tx + 16q) of the block and of the
// forward-substitution state S (initially I) in registers.  Column j of the factor is final once columns
// 0..j-1 have been eliminated, and so is row j of S; one iteration publishes both (unscaled), then every thread
// applies  A[i][c] -= L[i][j] L[c][j]  and  S[i][c] -= L[i][j] X[j][c]  with  X[j][:] = S[j][:] / L[j][j]
// to its own elements: one barrier per column (the two publish buffers alternate).  The columns are taken in
// three groups of 16 (JB), so that which sub-grid elements are above, on or below row / column j is known at
// compile time except for the group that holds j itself.
template <int JB>
__device__ __forceinline__ void chol_diag_columns(double (&a)[3][3], double (&s)[3][3], double (*colL)[NB],
                                                  double (*rowS)[NB], int nb, int k0, int32_t* info) {
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int jend = min(16, nb - 16 * JB);
    for (int jl = 0; jl < jend; ++jl) {
        const int j = 16 * JB + jl;
        double* cl = colL[jl & 1];
        double* rs = rowS[jl & 1];
        if (tx == jl) {
#pragma unroll
            for (int p = JB; p < 3; ++p) cl[ty + 16 * p] = a[p][JB];
        }
        if (ty == jl) {
#pragma unroll
            for (int q = 0; q <= JB; ++q) rs[tx + 16 * q] = s[JB][q];
        }
        __syncthreads();
        const double piv = cl[j];
        double ljj = 1.0, inv = 1.0;         // every thread scales by the same reciprocal: FP64 divisions are scarce
        if (!(piv > 0.0) || !isfinite(piv)) {
            if (tid == 0) atomicCAS(info, 0, 1 + k0 + j);
        } else {
            inv = rsqrt(piv);
            ljj = piv * inv;
        }
        double li[3], lc[3], xr[3];
#pragma unroll
        for (int p = JB; p < 3; ++p) li[p] = cl[ty + 16 * p] * inv;
#pragma unroll
        for (int q = JB; q < 3; ++q) lc[q] = cl[tx + 16 * q] * inv;
#pragma unroll
        for (int q = 0; q <= JB; ++q) xr[q] = rs[tx + 16 * q] * inv;
        const bool row_on = ty == jl, row_below = ty > jl, col_on = tx == jl, col_right = tx > jl;
#pragma unroll
        for (int p = JB; p < 3; ++p) {
            const bool below = p > JB || row_below;            // row i > j
            const bool on = p == JB && row_on;                 // row i == j
#pragma unroll
            for (int q = JB; q <= p; ++q) {                    // factor: columns c >= j of rows i >= j
                const bool right = q > JB || col_right;
                const bool oncol = q == JB && col_on;
                if (below && right) a[p][q] = fma(-li[p], lc[q], a[p][q]);
                else if (below && oncol) a[p][q] = li[p];
                else if (on && oncol) a[p][q] = ljj;
            }
#pragma unroll
            for (int q = 0; q <= JB; ++q) {                    // substitution: X[j][c] is zero for c > j
                if (below) s[p][q] = fma(-li[p], xr[q], s[p][q]);
                else if (on) s[p][q] = xr[q];
            }
        }
    }
}

__global__ void __launch_bounds__(256) chol_diag_kernel(double* __restrict__ A, double* __restrict__ Li, int d, int k0,
                                                        int nb, int32_t* info) {
    static_assert(NB == 48, "3 x 3 elements per thread of a 16 x 16 thread grid");
    __shared__ double colL[2][NB];
    __shared__ double rowS[2][NB];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    double a[3][3], s[3][3];
#pragma unroll
    for (int p = 0; p < 3; ++p)
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            const int i = ty + 16 * p, c = tx + 16 * q;
            a[p][q] = (i < nb && c <= i) ? A[(size_t)(k0 + i) * d + k0 + c] : 0.0;
            s[p][q] = i == c ? 1.0 : 0.0;
        }
    chol_diag_columns<0>(a, s, colL, rowS, nb, k0, info);
    if (nb > 16) chol_diag_columns<1>(a, s, colL, rowS, nb, k0, info);
    if (nb > 32) chol_diag_columns<2>(a, s, colL, rowS, nb, k0, info);
#pragma unroll
    for (int p = 0; p < 3; ++p)
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            const int i = ty + 16 * p, c = tx + 16 * q;
            if (i < nb && c < nb) {
                if (c <= i) A[(size_t)(k0 + i) * d + k0 + c] = a[p][q];
                Li[(size_t)(k0 + i) * d + k0 + c] = c <= i ? s[p][q] : 0.0;
            }
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
            // panel below the diagonal block: A21 <- A21 * inv(L11)^T, in place
            double* P = A + (size_t)(k0 + nb) * d + k0;
            dgemm<false, true>(s, below, nb, nb, 1.0, P, d, Li + (size_t)k0 * d + k0, d, 0.0, P, d);
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
