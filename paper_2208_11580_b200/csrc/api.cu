// C ABI of the OBC library: argument checks on the host (nothing is launched or written when they fail),
// then dispatch to the kernels.  See include/obc.h for the contract of every entry point.
#include "engine.cuh"
#include <atomic>
#include <mutex>

namespace obc {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

obc_status device_info(DeviceInfo* out) {
    static std::mutex mu;
    static DeviceInfo cache[64];
    static bool have[64] = {};
    int dev = 0;
    OBC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return OBC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!have[dev]) {
        DeviceInfo di;
        OBC_CUDA_TRY(cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev));
        OBC_CUDA_TRY(cudaDeviceGetAttribute(&di.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        OBC_CUDA_TRY(cudaDeviceGetAttribute(&di.l2_bytes, cudaDevAttrL2CacheSize, dev));
        cache[dev] = di;
        have[dev] = true;
    }
    *out = cache[dev];
    return OBC_OK;
}

// Validates the caller's per-call engine options (NULL = defaults) and copies them.
static bool engine_opts_ok(const obc_engine_opts* o, EngineOpts* out) {
    out->engine = OBC_ENGINE_AUTO; out->threads = 0; out->max_pending = 0; out->flags = 0;
    if (!o) return true;
    if (o->engine != OBC_ENGINE_AUTO && o->engine != OBC_ENGINE_STREAMING && o->engine != OBC_ENGINE_BLOCKED) return false;
    if (o->threads != 0 && o->threads != 128 && o->threads != 256 && o->threads != 512) return false;
    if (o->max_pending < 0 || o->max_pending > 64 || (o->flags & ~OBC_ENGINE_WHOLE_WAVES)) return false;
    out->engine = o->engine; out->threads = o->threads; out->max_pending = o->max_pending; out->flags = o->flags;
    return true;
}

static bool mat_ok(const void* p, int64_t ld, int64_t min_ld) { return p && ld >= min_ld; }
static bool mat_aligned(const void* p, int64_t ld) { return aligned16(p) && (ld % 4 == 0); }
static bool rows_ok(int d_row, int d_col, int row_begin, int row_count) {
    return d_row > 0 && d_col > 0 && row_begin >= 0 && row_count > 0 && (int64_t)row_begin + row_count <= d_row;
}

}  // namespace obc

using namespace obc;

extern "C" {

const char* obc_status_string(obc_status s) {
    switch (s) {
        case OBC_OK: return "ok";
        case OBC_ERR_INVALID_ARG: return "invalid argument";
        case OBC_ERR_ALIGNMENT: return "pointer or leading dimension not aligned";
        case OBC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case OBC_ERR_NOT_POSDEF: return "Hessian not positive definite";
        case OBC_ERR_NONFINITE: return "non-positive or non-finite inverse-Hessian diagonal";
        case OBC_ERR_TIMEOUT: return "device-side wait timed out";
        case OBC_ERR_CUDA: return "CUDA runtime error";
        case OBC_ERR_UNSUPPORTED: return "size not supported";
        case OBC_ERR_STATIC_SCRATCH: return "problem exceeds the built-in scratch area of this allocation-free entry point";
    }
    return "unknown status";
}

unsigned long long obc_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

obc_status obc_engine_plan(int d_col, int with_trace, int row_count, const obc_engine_opts* opts, int32_t* plan) {
    EngineOpts eo;
    if (d_col <= 0 || row_count < 0 || !plan || !engine_opts_ok(opts, &eo)) return OBC_ERR_INVALID_ARG;
    if (eo.engine == OBC_ENGINE_STREAMING) return streaming_engine_plan(d_col, plan);
    return blocked_engine_plan(d_col, with_trace, row_count, eo, plan);
}

size_t obc_workspace_bytes(obc_op op, int row_count, int d_col, int64_t n) {
    if (d_col <= 0 || row_count < 0) return 0;
    switch (op) {
        case OBC_OP_HESSIAN: return n > 0 ? hessian_workspace_bytes(d_col, n) : 0;
        case OBC_OP_INVERSE: return inverse_workspace_bytes(d_col);
        case OBC_OP_SELECT: return row_count > 0 ? select_workspace_bytes(row_count, d_col) : 0;
        case OBC_OP_CROSS_GRAM: return (n > 0 && row_count > 0) ? cross_workspace_bytes(row_count, d_col, n) : 0;
        case OBC_OP_REFIT: return row_count > 0 ? cross_workspace_bytes(row_count, d_col, d_col) : 0;
        case OBC_OP_PRUNE_BLOCKS: {
            DeviceInfo di;
            if (device_info(&di) != OBC_OK || d_col > OBC_MAX_DCOL) return 0;
            return engine_blocks_workspace_bytes(row_count, d_col, di);
        }
        case OBC_OP_PRUNE_TRACE:
        case OBC_OP_PRUNE_APPLY:
        case OBC_OP_QUANTIZE: {
            DeviceInfo di;
            if (device_info(&di) != OBC_OK || d_col > OBC_MAX_DCOL) return 0;
            return engine_workspace_bytes(row_count, d_col, di);
        }
    }
    return 0;
}

obc_status obc_hessian(const float* X, int d_col, int64_t n, int64_t ldx, float* H, int ldh, int accumulate,
                       obc_prec prec, int32_t* info, int wait_limit, void* ws, size_t ws_bytes, obc_stream stream) {
    if (d_col <= 0 || n <= 0 || !mat_ok(X, ldx, n) || !mat_ok(H, ldh, d_col)) return OBC_ERR_INVALID_ARG;
    if (accumulate != 0 && accumulate != 1) return OBC_ERR_INVALID_ARG;
    if (prec != OBC_PREC_FP32 && prec != OBC_PREC_TF32 && prec != OBC_PREC_BF16X3) return OBC_ERR_INVALID_ARG;
    if (!mat_aligned(X, ldx) || !mat_aligned(H, ldh)) return OBC_ERR_ALIGNMENT;
    if (!ws || !aligned256(ws) || ws_bytes < hessian_workspace_bytes(d_col, n)) return OBC_ERR_WORKSPACE;
    if (prec == OBC_PREC_FP32) return hessian_fp32_launch(X, d_col, n, ldx, H, ldh, accumulate, info, ws, (cudaStream_t)stream);
    return hessian_tc_launch(X, d_col, n, ldx, H, ldh, accumulate, prec, info, wait_limit, ws, (cudaStream_t)stream);
}

obc_status obc_cross_gram(const float* Y, int64_t ldy, const float* X, int64_t ldx, int d_row, int d_col, int64_t n,
                          float* G, int ldg, int accumulate, obc_prec prec, int32_t* info, int wait_limit, void* ws,
                          size_t ws_bytes, obc_stream stream) {
    if (d_row <= 0 || d_col <= 0 || n <= 0 || !mat_ok(Y, ldy, n) || !mat_ok(X, ldx, n) || !mat_ok(G, ldg, d_col))
        return OBC_ERR_INVALID_ARG;
    if (accumulate != 0 && accumulate != 1) return OBC_ERR_INVALID_ARG;
    if (prec != OBC_PREC_FP32 && prec != OBC_PREC_TF32 && prec != OBC_PREC_BF16X3) return OBC_ERR_INVALID_ARG;
    if (!mat_aligned(Y, ldy) || !mat_aligned(X, ldx)) return OBC_ERR_ALIGNMENT;
    if (prec == OBC_PREC_FP32) {
        if (info) OBC_CUDA_TRY(cudaMemsetAsync(info, 0, sizeof(int32_t), (cudaStream_t)stream));   // this path has no waits
        return sgemm_nt_launch(d_row, d_col, n, 1.f, Y, ldy, X, ldx, accumulate ? 1.f : 0.f, G, ldg, (cudaStream_t)stream);
    }
    if (!ws || !aligned256(ws) || ws_bytes < cross_workspace_bytes(d_row, d_col, n)) return OBC_ERR_WORKSPACE;
    return cross_tc_launch(Y, d_row, ldy, X, d_col, ldx, n, G, ldg, accumulate, 1.f, prec, info, wait_limit, ws,
                           (cudaStream_t)stream);
}

obc_status obc_refit(const float* G, int ldg, const float* Hinv, int ldhi, int d_row, int d_col, float* W_out, int ldwo,
                     obc_prec prec, void* ws, size_t ws_bytes, obc_stream stream) {
    if (d_row <= 0 || d_col <= 0 || !mat_ok(G, ldg, d_col) || !mat_ok(Hinv, ldhi, d_col) || !mat_ok(W_out, ldwo, d_col))
        return OBC_ERR_INVALID_ARG;
    if (prec != OBC_PREC_FP32 && prec != OBC_PREC_TF32 && prec != OBC_PREC_BF16X3) return OBC_ERR_INVALID_ARG;
    // Hinv is symmetric, so G Hinv = G Hinv^T is the "A B^T" product (contraction over d_col)
    if (prec == OBC_PREC_FP32)
        return sgemm_nt_launch(d_row, d_col, d_col, 2.f, G, ldg, Hinv, ldhi, 0.f, W_out, ldwo, (cudaStream_t)stream);
    if (!mat_aligned(G, ldg) || !mat_aligned(Hinv, ldhi)) return OBC_ERR_ALIGNMENT;
    if (!ws || !aligned256(ws) || ws_bytes < cross_workspace_bytes(d_row, d_col, d_col)) return OBC_ERR_WORKSPACE;
    return cross_tc_launch(G, d_row, ldg, Hinv, d_col, ldhi, d_col, W_out, ldwo, 0, 2.f, prec, nullptr, 0, ws,
                           (cudaStream_t)stream);
}

obc_status obc_hessian_inverse(const float* H, int d_col, int ldh, float damp_rel, float* Hinv, int ldhi,
                               int32_t* info, void* ws, size_t ws_bytes, obc_stream stream) {
    if (d_col <= 0 || !mat_ok(H, ldh, d_col) || !mat_ok(Hinv, ldhi, d_col) || !info) return OBC_ERR_INVALID_ARG;
    if (!(damp_rel >= 0.f)) return OBC_ERR_INVALID_ARG;
    if (!mat_aligned(H, ldh) || !mat_aligned(Hinv, ldhi)) return OBC_ERR_ALIGNMENT;
    if (!ws || !aligned256(ws) || ws_bytes < inverse_workspace_bytes(d_col)) return OBC_ERR_WORKSPACE;
    return inverse_launch(H, d_col, ldh, damp_rel, Hinv, ldhi, info, ws, (cudaStream_t)stream);
}

obc_status obc_prune_trace(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                           const float* Hinv, int ldhi, int steps, int32_t* order, float* loss, float* w_trace,
                           int32_t* row_status, void* ws, size_t ws_bytes, const obc_engine_opts* opts, obc_stream stream) {
    EngineOpts eo;
    if (!engine_opts_ok(opts, &eo)) return OBC_ERR_INVALID_ARG;
    if (!rows_ok(d_row, d_col, row_begin, row_count) || !mat_ok(W, ldw, d_col) || !mat_ok(Hinv, ldhi, d_col))
        return OBC_ERR_INVALID_ARG;
    if (steps < 1 || steps > d_col || !order || !loss || !row_status) return OBC_ERR_INVALID_ARG;
    if (d_col > OBC_MAX_DCOL) return OBC_ERR_UNSUPPORTED;
    if (!mat_aligned(W, ldw) || !mat_aligned(Hinv, ldhi)) return OBC_ERR_ALIGNMENT;
    return engine_prune_trace(W, ldw, d_row, d_col, row_begin, row_count, Hinv, ldhi, steps, order, loss, w_trace,
                              row_status, ws, ws_bytes, eo, (cudaStream_t)stream);
}

obc_status obc_prune_nm(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                        const float* Hinv, int ldhi, int n_keep, int m_block, int32_t* order, float* loss,
                        float* W_out, int ldwo, uint8_t* mask, int32_t* row_status, void* ws, size_t ws_bytes,
                        const obc_engine_opts* opts, obc_stream stream) {
    EngineOpts eo;
    if (!engine_opts_ok(opts, &eo)) return OBC_ERR_INVALID_ARG;
    if (!rows_ok(d_row, d_col, row_begin, row_count) || !mat_ok(W, ldw, d_col) || !mat_ok(Hinv, ldhi, d_col))
        return OBC_ERR_INVALID_ARG;
    if (!mat_ok(W_out, ldwo, d_col) || !row_status) return OBC_ERR_INVALID_ARG;
    if (m_block != 2 && m_block != 4 && m_block != 8 && m_block != 16 && m_block != 32) return OBC_ERR_INVALID_ARG;
    if (n_keep <= 0 || n_keep >= m_block || d_col % m_block != 0) return OBC_ERR_INVALID_ARG;
    if (d_col > OBC_MAX_DCOL) return OBC_ERR_UNSUPPORTED;
    if (!mat_aligned(W, ldw) || !mat_aligned(Hinv, ldhi)) return OBC_ERR_ALIGNMENT;
    return engine_prune_nm(W, ldw, d_row, d_col, row_begin, row_count, Hinv, ldhi, n_keep, m_block, order, loss, W_out,
                           ldwo, mask, row_status, ws, ws_bytes, eo, (cudaStream_t)stream);
}

obc_status obc_prune_blocks(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                            const float* Hinv, int ldhi, int block, int32_t* order, float* loss, float* w_trace,
                            int32_t* row_status, void* ws, size_t ws_bytes, const obc_engine_opts* opts, obc_stream stream) {
    EngineOpts eo;
    if (!engine_opts_ok(opts, &eo)) return OBC_ERR_INVALID_ARG;
    if (!rows_ok(d_row, d_col, row_begin, row_count) || !mat_ok(W, ldw, d_col) || !mat_ok(Hinv, ldhi, d_col))
        return OBC_ERR_INVALID_ARG;
    if (!order || !loss || !row_status || block <= 0 || d_col % block != 0) return OBC_ERR_INVALID_ARG;
    if ((block != 4 && block != 8) || d_col > OBC_MAX_DCOL) return OBC_ERR_UNSUPPORTED;
    if (!mat_aligned(W, ldw) || !mat_aligned(Hinv, ldhi)) return OBC_ERR_ALIGNMENT;
    return engine_prune_blocks(W, ldw, d_row, d_col, row_begin, row_count, Hinv, ldhi, block, order, loss, w_trace,
                               row_status, ws, ws_bytes, eo, (cudaStream_t)stream);
}

obc_status obc_select_global_mask(const float* loss, const int32_t* order, int d_row, int d_col, int64_t k,
                                  int32_t* counts, uint8_t* mask, void* ws, size_t ws_bytes, obc_stream stream) {
    if (d_row <= 0 || d_col <= 0 || !loss || !order || !counts || !mask) return OBC_ERR_INVALID_ARG;
    if (k < 0 || k > (int64_t)d_row * d_col) return OBC_ERR_INVALID_ARG;
    if (!ws || !aligned256(ws) || ws_bytes < select_workspace_bytes(d_row, d_col)) return OBC_ERR_WORKSPACE;
    return select_launch(loss, order, d_row, d_col, k, counts, mask, ws, (cudaStream_t)stream);
}

obc_status obc_prune_apply(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                           const float* Hinv, int ldhi, const int32_t* order, const int32_t* counts,
                           const float* w_trace, int trace_steps, float* W_out, int ldwo, int32_t* row_status,
                           void* ws, size_t ws_bytes, const obc_engine_opts* opts, obc_stream stream) {
    EngineOpts eo;
    if (!engine_opts_ok(opts, &eo)) return OBC_ERR_INVALID_ARG;
    if (!rows_ok(d_row, d_col, row_begin, row_count) || !counts || !mat_ok(W_out, ldwo, d_col))
        return OBC_ERR_INVALID_ARG;
    if (w_trace) {
        if (trace_steps < 1 || trace_steps > d_col) return OBC_ERR_INVALID_ARG;
        return trace_gather_launch(w_trace, trace_steps, counts, d_col, row_begin, row_count, W_out, ldwo,
                                   (cudaStream_t)stream);
    }
    if (!mat_ok(W, ldw, d_col) || !mat_ok(Hinv, ldhi, d_col) || !order || !row_status) return OBC_ERR_INVALID_ARG;
    if (d_col > OBC_MAX_DCOL) return OBC_ERR_UNSUPPORTED;
    if (!mat_aligned(W, ldw) || !mat_aligned(Hinv, ldhi)) return OBC_ERR_ALIGNMENT;
    return engine_replay(W, ldw, d_row, d_col, row_begin, row_count, Hinv, ldhi, order, counts, W_out, ldwo,
                         row_status, ws, ws_bytes, eo, (cudaStream_t)stream);
}

obc_status obc_minmax_grid(const float* W, int ldw, int d_row, int d_col, const uint8_t* mask, int bits,
                           int symmetric, float* scale, float* zero, int* maxq_host, obc_stream stream) {
    if (d_row <= 0 || d_col <= 0 || !mat_ok(W, ldw, d_col) || !scale || !zero) return OBC_ERR_INVALID_ARG;
    if (bits < 2 || bits > 16 || (symmetric != 0 && symmetric != 1)) return OBC_ERR_INVALID_ARG;
    if (maxq_host) *maxq_host = grid_maxq(bits, symmetric);
    return minmax_grid_launch(W, ldw, d_row, d_col, mask, bits, symmetric, scale, zero, (cudaStream_t)stream);
}

obc_status obc_quantize(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                        const float* Hinv, int ldhi, float* scale, float* zero, int bits, int symmetric,
                        const int32_t* prune_order, const int32_t* prune_counts, int flags, float* W_out, int ldwo,
                        int32_t* codes, float* loss, int32_t* qorder, int32_t* row_status, void* ws,
                        size_t ws_bytes, const obc_engine_opts* opts, obc_stream stream) {
    EngineOpts eo;
    if (!engine_opts_ok(opts, &eo)) return OBC_ERR_INVALID_ARG;
    if (!rows_ok(d_row, d_col, row_begin, row_count) || !mat_ok(W, ldw, d_col) || !mat_ok(Hinv, ldhi, d_col))
        return OBC_ERR_INVALID_ARG;
    if (!scale || !zero || !mat_ok(W_out, ldwo, d_col) || !codes || !row_status) return OBC_ERR_INVALID_ARG;
    if (bits < 2 || bits > 16 || (symmetric != 0 && symmetric != 1)) return OBC_ERR_INVALID_ARG;
    if ((prune_order == nullptr) != (prune_counts == nullptr)) return OBC_ERR_INVALID_ARG;
    if (flags & ~OBC_FLAG_OUTLIERS) return OBC_ERR_INVALID_ARG;
    if (d_col > OBC_MAX_DCOL) return OBC_ERR_UNSUPPORTED;
    if (!mat_aligned(W, ldw) || !mat_aligned(Hinv, ldhi)) return OBC_ERR_ALIGNMENT;
    return engine_quantize(W, ldw, d_row, d_col, row_begin, row_count, Hinv, ldhi, scale, zero, bits, symmetric,
                           prune_order, prune_counts, flags, W_out, ldwo, codes, loss, qorder, row_status, ws,
                           ws_bytes, eo, (cudaStream_t)stream);
}

}  // extern "C"
