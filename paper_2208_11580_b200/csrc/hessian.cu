// Layer Hessian H = 2 X X^T (Section 3 of "Optimal Brain Compression": Hessian of each row's least-squares
// problem; identical for all rows; further calibration chunks are accumulated into it).
//
// X is d x n with the calibration axis contiguous, so both GEMM operands are K-major.  Only tiles on or
// below the diagonal are computed (SYRK); the calibration axis is split into slices whose partial sums are
// combined in a fixed order by the finalize kernel, which also applies the factor 2, mirrors the lower
// triangle (exactly symmetric output) and adds to the previous H when accumulating.  Deterministic.
//
// This file holds the FP32 CUDA-core path (OBC_PREC_FP32), the slice/finalize machinery, and the dispatch
// to the tensor-core paths.
#include "common.cuh"

namespace obc {

constexpr int HT = 128;           // output tile
constexpr int HK = 16;            // k chunk

int hessian_splits(int d, int64_t n) {
    const int T = (d + HT - 1) / HT;
    const int ntiles = T * (T + 1) / 2;
    int64_t s = (444 + ntiles - 1) / ntiles;
    const int64_t by_len = (n + 2047) / 2048;      // short accumulation chains: partial sums are combined in FP32 RN
    if (by_len > s) s = by_len;
    if (s > 32) s = 32;
    if (s * 64 > n) s = n / 64;
    if (s < 1) s = 1;
    return (int)s;
}

size_t hessian_tc_extra_bytes(int d, int64_t n);

size_t hessian_workspace_bytes(int d, int64_t n) {      // partial sums + what the tensor-core paths add
    return round_up((size_t)hessian_splits(d, n) * d * d * sizeof(float), 256) + hessian_tc_extra_bytes(d, n);
}

// partial[z][i][j] = sum_{k in slice z} X[i][k] X[j][k]   for tiles with bj <= bi
__global__ void __launch_bounds__(256) syrk_fp32_kernel(const float* __restrict__ X, int d, int64_t n, int64_t ldx,
                                                        int64_t slice, float* __restrict__ partial) {
    // blockIdx.x enumerates lower-triangular tile pairs
    int bi = 0, t = blockIdx.x;
    while (t > bi) { t -= bi + 1; ++bi; }
    const int bj = t;
    const int64_t kb = (int64_t)blockIdx.y * slice;
    const int64_t ke = kb + slice < n ? kb + slice : n;
    __shared__ __align__(16) float As[HK][HT + 4];
    __shared__ __align__(16) float Bs[HK][HT + 4];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    float acc[8][8] = {};
    const bool vec_ok = (ldx % 4 == 0) && ((reinterpret_cast<uintptr_t>(X) & 15u) == 0) && (kb % 4 == 0);
    for (int64_t k0 = kb; k0 < ke; k0 += HK) {
#pragma unroll
        for (int rep = 0; rep < 2; ++rep) {
            const int q = tid + rep * 256;
            const int row = q >> 2, kq = (q & 3) * 4;
            const int64_t k = k0 + kq;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const int gi = (which ? bj : bi) * HT + row;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (gi < d) {
                    const float* src = X + (size_t)gi * ldx + k;
                    if (vec_ok && k + 3 < ke) v = *reinterpret_cast<const float4*>(src);
                    else {
                        if (k + 0 < ke) v.x = src[0];
                        if (k + 1 < ke) v.y = src[1];
                        if (k + 2 < ke) v.z = src[2];
                        if (k + 3 < ke) v.w = src[3];
                    }
                }
                float(*S)[HT + 4] = which ? Bs : As;
                S[kq + 0][row] = v.x; S[kq + 1][row] = v.y; S[kq + 2][row] = v.z; S[kq + 3][row] = v.w;
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < HK; ++k) {
            const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
            const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* P = partial + (size_t)blockIdx.y * d * d;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int gi = bi * HT + (i < 4 ? ty * 4 + i : 64 + ty * 4 + i - 4);
        if (gi >= d) continue;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int gj = bj * HT + (j < 4 ? tx * 4 + j : 64 + tx * 4 + j - 4);
            if (gj < d) P[(size_t)gi * d + gj] = acc[i][j];
        }
    }
}

// H[i][j] = H[j][i] = (accumulate ? H[i][j] : 0) + 2 * sum_z partial[z][i][j]     for j <= i
// err (nullable): a non-zero flag from the producing kernel (a bounded wait that expired) turns the whole result
// into NaN; info (nullable) receives 0 or OBC_ERR_TIMEOUT accordingly.
__global__ void __launch_bounds__(256) hessian_finalize_kernel(const float* __restrict__ partial, int splits, int d,
                                                               float* __restrict__ H, int ldh, int accumulate,
                                                               const int* __restrict__ err, int32_t* __restrict__ info) {
    const int i = blockIdx.y;
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (info && i == 0 && j == 0) info[0] = (err && *err != 0) ? (int32_t)OBC_ERR_TIMEOUT : 0;
    if (j > i || j >= d) return;
    float s = 0.f;
    for (int z = 0; z < splits; ++z) s += partial[(size_t)z * d * d + (size_t)i * d + j];
    float v = 2.f * s;
    if (accumulate) v += H[(size_t)i * ldh + j];
    if (err && *err != 0) v = __int_as_float(0x7fc00000);
    H[(size_t)i * ldh + j] = v;
    H[(size_t)j * ldh + i] = v;
}

obc_status hessian_finalize_launch(const float* partial, int splits, int d, float* H, int ldh, int accumulate,
                                   const int* err, int32_t* info, cudaStream_t stream) {
    dim3 grid((d + 255) / 256, d);
    hessian_finalize_kernel<<<grid, 256, 0, stream>>>(partial, splits, d, H, ldh, accumulate, err, info);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

obc_status hessian_fp32_launch(const float* X, int d, int64_t n, int64_t ldx, float* H, int ldh, int accumulate,
                               int32_t* info, void* ws, cudaStream_t stream) {
    const int splits = hessian_splits(d, n);
    int64_t slice = (n + splits - 1) / splits;
    slice = (slice + HK - 1) / HK * HK;
    const int T = (d + HT - 1) / HT;
    dim3 grid(T * (T + 1) / 2, splits);
    float* partial = reinterpret_cast<float*>(ws);
    syrk_fp32_kernel<<<grid, 256, 0, stream>>>(X, d, n, ldx, slice, partial);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return hessian_finalize_launch(partial, splits, d, H, ldh, accumulate, nullptr, info, stream);
}

}  // namespace obc
