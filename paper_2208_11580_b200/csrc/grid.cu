// Per-row min-max quantisation grid over the kept weights, and the trace gather of the "more memory"
// reconstruction option (Figure 1 of "Optimal Brain Compression").
#include "common.cuh"

namespace obc {

constexpr int GRID_THREADS = 256;

__global__ void __launch_bounds__(GRID_THREADS) minmax_grid_kernel(const float* __restrict__ W, int ldw, int d,
                                                                   const uint8_t* __restrict__ mask, int bits,
                                                                   int symmetric, float* __restrict__ scale,
                                                                   float* __restrict__ zero) {
    __shared__ float slo[GRID_THREADS], shi[GRID_THREADS];
    const int r = blockIdx.x;
    float lo = 0.f, hi = 0.f;
    for (int j = threadIdx.x; j < d; j += GRID_THREADS) {
        if (mask && !mask[(size_t)r * d + j]) continue;
        const float w = W[(size_t)r * ldw + j];
        lo = fminf(lo, w);
        hi = fmaxf(hi, w);
    }
    slo[threadIdx.x] = lo; shi[threadIdx.x] = hi;
    __syncthreads();
    for (int off = GRID_THREADS / 2; off; off >>= 1) {
        if (threadIdx.x < off) {
            slo[threadIdx.x] = fminf(slo[threadIdx.x], slo[threadIdx.x + off]);
            shi[threadIdx.x] = fmaxf(shi[threadIdx.x], shi[threadIdx.x + off]);
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) grid_from_range(slo[0], shi[0], bits, symmetric, &scale[r], &zero[r]);
}

// W_out[r][:] = w_trace[r][counts[r]][:]      one block per row
__global__ void __launch_bounds__(GRID_THREADS) trace_gather_kernel(const float* __restrict__ w_trace, int trace_steps,
                                                                    const int32_t* __restrict__ counts, int d,
                                                                    int row_begin, float* __restrict__ W_out, int ldwo) {
    const int r = row_begin + blockIdx.x;
    int c = counts[r];
    c = c < 0 ? 0 : (c > trace_steps ? trace_steps : c);
    const float* src = w_trace + ((size_t)r * (trace_steps + 1) + c) * d;
    for (int j = threadIdx.x; j < d; j += GRID_THREADS) W_out[(size_t)r * ldwo + j] = src[j];
}

obc_status minmax_grid_launch(const float* W, int ldw, int rows, int d, const uint8_t* mask, int bits, int symmetric,
                              float* scale, float* zero, cudaStream_t stream) {
    minmax_grid_kernel<<<rows, GRID_THREADS, 0, stream>>>(W, ldw, d, mask, bits, symmetric, scale, zero);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

obc_status trace_gather_launch(const float* w_trace, int trace_steps, const int32_t* counts, int d, int row_begin,
                               int row_count, float* W_out, int ldwo, cudaStream_t stream) {
    trace_gather_kernel<<<row_count, GRID_THREADS, 0, stream>>>(w_trace, trace_steps, counts, d, row_begin, W_out, ldwo);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

}  // namespace obc
