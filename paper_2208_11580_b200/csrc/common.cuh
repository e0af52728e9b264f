// Shared host/device helpers of the OBC CUDA library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>
#include "obc.h"

#define OBC_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) return OBC_ERR_CUDA;         \
    } while (0)

namespace obc {

// Every kernel launch of the library goes through this counter (read by obc_kernel_launches()).
void count_launch(int n = 1);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Properties of the current device, queried once per device and cached (host side only).
struct DeviceInfo {
    int sm_count;
    int smem_optin;   // max dynamic shared memory per block (opt-in), bytes
    int l2_bytes;
};
obc_status device_info(DeviceInfo* out);

// maxq of the uniform grid for (bits, symmetric)
__host__ __device__ inline int grid_maxq(int bits, int symmetric) {
    return symmetric ? 2 * ((1 << (bits - 1)) - 1) : (1 << bits) - 1;
}

// The per-row min-max grid rule, in FP32, shared by the grid kernel and the compound path of the row
// engine so that both produce identical parameters from identical (lo, hi).
__host__ __device__ inline void grid_from_range(float lo, float hi, int bits, int symmetric,
                                                float* scale, float* zero) {
    lo = lo < 0.f ? lo : 0.f;
    hi = hi > 0.f ? hi : 0.f;
    if (symmetric) {
        const float Q = (float)((1 << (bits - 1)) - 1);
        const float a = hi > -lo ? hi : -lo;
        *scale = a > 0.f ? a / Q : 1.f;
        *zero = Q;
    } else {
        const float mq = (float)((1 << bits) - 1);
        const float sc = hi > lo ? (hi - lo) / mq : 1.f;
        *scale = sc;
#ifdef __CUDA_ARCH__
        *zero = rintf(-lo / sc);
#else
        *zero = __builtin_rintf(-lo / sc);
#endif
    }
}

// The per-call engine options of obc_engine_opts after validation (all zero = defaults).
struct EngineOpts { int engine; int threads; int max_pending; int flags; };

// ---- launchers implemented in the kernel files --------------------------------------------------------------
size_t engine_workspace_bytes(int row_count, int d, const DeviceInfo& di);
size_t select_workspace_bytes(int rows, int d);
size_t inverse_workspace_bytes(int d);
size_t hessian_workspace_bytes(int d, int64_t n);
obc_status select_launch(const float* loss, const int32_t* order, int rows, int d, int64_t k, int32_t* counts,
                         uint8_t* mask, void* ws, cudaStream_t stream);
obc_status inverse_launch(const float* H, int d, int ldh, float damp_rel, float* Hinv, int ldhi, int32_t* info,
                          void* ws, cudaStream_t s);
obc_status hessian_fp32_launch(const float* X, int d, int64_t n, int64_t ldx, float* H, int ldh, int accumulate,
                               int32_t* info, void* ws, cudaStream_t stream);
obc_status hessian_tc_launch(const float* X, int d, int64_t n, int64_t ldx, float* H, int ldh, int accumulate,
                             obc_prec prec, int32_t* info, int wait_limit, void* ws, cudaStream_t stream);
size_t cross_workspace_bytes(int rows_a, int rows_b, int64_t n);
obc_status cross_tc_launch(const float* Y, int rows_a, int64_t ldy, const float* X, int rows_b, int64_t ldx, int64_t n,
                           float* G, int ldg, int accumulate, float alpha, obc_prec prec, int32_t* info, int wait_limit,
                           void* ws, cudaStream_t stream);
obc_status sgemm_nt_launch(int M, int N, int64_t K, float alpha, const float* A, int64_t lda, const float* B, int64_t ldb,
                           float beta, float* C, int ldc, cudaStream_t stream);
obc_status minmax_grid_launch(const float* W, int ldw, int rows, int d, const uint8_t* mask, int bits, int symmetric,
                              float* scale, float* zero, cudaStream_t stream);
obc_status trace_gather_launch(const float* w_trace, int trace_steps, const int32_t* counts, int d, int row_begin,
                               int row_count, float* W_out, int ldwo, cudaStream_t stream);
obc_status engine_prune_trace(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                              const float* Hinv, int ldhi, int steps, int32_t* order, float* loss, float* w_trace,
                              int32_t* row_status, void* ws, size_t ws_bytes, const EngineOpts& eo, cudaStream_t stream);
obc_status engine_prune_nm(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                           const float* Hinv, int ldhi, int n_keep, int m_block, int32_t* order, float* loss,
                           float* W_out, int ldwo, uint8_t* mask, int32_t* row_status, void* ws, size_t ws_bytes,
                           const EngineOpts& eo, cudaStream_t stream);
obc_status engine_prune_blocks(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                               const float* Hinv, int ldhi, int block, int32_t* order, float* loss, float* w_trace,
                               int32_t* row_status, void* ws, size_t ws_bytes, const EngineOpts& eo, cudaStream_t stream);
size_t engine_blocks_workspace_bytes(int row_count, int d, const DeviceInfo& di);
obc_status engine_replay(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                         const float* Hinv, int ldhi, const int32_t* order, const int32_t* counts, float* W_out,
                         int ldwo, int32_t* row_status, void* ws, size_t ws_bytes, const EngineOpts& eo, cudaStream_t stream);
obc_status engine_quantize(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                           const float* Hinv, int ldhi, float* scale, float* zero, int bits, int symmetric,
                           const int32_t* prune_order, const int32_t* prune_counts, int flags, float* W_out,
                           int ldwo, int32_t* codes, float* loss, int32_t* qorder, int32_t* row_status, void* ws,
                           size_t ws_bytes, const EngineOpts& eo, cudaStream_t stream);

}  // namespace obc
