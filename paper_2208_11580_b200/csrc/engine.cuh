// Definitions shared by the two row elimination engines (Algorithm 1 / Algorithm 3 of "Optimal Brain
// Compression"): the argument block, the per-step broadcast record, the grid function and the key order of
// the argmin.  row_engine.cu holds the streaming engine (one Lemma-1 pass over the row's matrix per step),
// row_engine_blocked.cu the engine that defers the Lemma-1 updates and applies them several at a time.
#pragma once
#include "common.cuh"
#include <math_constants.h>

namespace obc {

enum EngineMode { MODE_PRUNE = 0, MODE_REPLAY = 1, MODE_QUANT = 2, MODE_REPLAY_QUANT = 3 };

struct EngineArgs {
    const float* W; int ldw;
    int d; int row_begin; int row_count;
    const float* Hinv; int ldhi;
    int mode; int steps;
    const int32_t* forced_order; const int32_t* forced_counts;
    float* scale; float* zero; int bits; int symmetric; int flags;
    int32_t* order; float* loss;
    float* w_trace; int trace_steps;
    float* W_out; int ldwo;
    int32_t* codes; int32_t* row_status;
    float* Hws; int ldp;                  // private triangles: gridDim.x blocks of d x ldp floats
    int ms;                               // on-chip threshold: finish in shared memory once m <= ms
    int cap;                              // d rounded up to a multiple of 4
    int panel_floats;                     // blocked engine: floats of shared memory for the pending vectors
    int max_pending;                      // blocked engine: upper limit on deferred updates (1..64)
    int nm_prune; int nm_lg;              // blocked engine, N:M pattern: at most nm_prune eliminations per block of
                                          // 2^nm_lg consecutive columns (nm_prune = 0: no pattern)
    uint8_t* mask;                        // blocked engine, nullable: d_row x d mask, 0 at eliminated columns
    int block_c;                          // blocked engine: 4 = block pruning in blocks of 4 columns (Eq. 5), 0 = off
    float* Gpan; int g_vectors; int g_ld; // blocked engine: overflow pending vectors in global memory (per block
                                          // g_vectors rows of g_ld floats), nullptr = none
    int split;                            // blocked engine: rows are shared out in equal work per block, a row may be
                                          // started by one block and finished by the next (see row_engine_blocked.cu)
    char* split_state; size_t split_stride;   // per block: saved state of the row it started for its neighbour
    int* split_flags;                     // per block: 1 once that state is complete (zeroed before the launch)
    EngineOpts opts;                      // the caller's per-call choice (host side only)
};

struct Bcast {                            // block-wide broadcast values, written by one thread
    double e, dpp, qp, code;
    double sc, ze, mq;
    int slot; int fail; int op; int nh;
};

__device__ __forceinline__ bool key_less(double s, int o, double s2, int o2) {
    return s < s2 || (s == s2 && o < o2);
}

// q(x) on the uniform grid; all FP64 so that the integer code is decided in the same precision as the
// FP64 reference decides it.
__device__ __forceinline__ double grid_q(double x, double sc, double ze, double mq, double* code) {
    double c = rint(x / sc) + ze;
    c = fmin(fmax(c, 0.0), mq);
    *code = c;
    return sc * (c - ze);
}

// Same result as grid_q with one multiplication instead of the division wherever the product x * (1/sc) is
// safely away from a rounding boundary (the two quotients differ by a few units in the last place at most);
// next to a boundary the true quotient decides, as in grid_q.
__device__ __forceinline__ double grid_q_fast(double x, double sc, double isc, double ze, double mq, double* code) {
    const double t = x * isc;
    double c = rint(t);
    if (fabs(fabs(t - c) - 0.5) < 1e-9 * fmax(1.0, fabs(t))) c = rint(x / sc);
    c = fmin(fmax(c + ze, 0.0), mq);
    *code = c;
    return sc * (c - ze);
}

// Launchers of the two engines (same arguments; each checks its own workspace need).
size_t streaming_engine_workspace_bytes(int row_count, int d, const DeviceInfo& di);
size_t blocked_engine_workspace_bytes(int row_count, int d, const DeviceInfo& di);
obc_status streaming_engine_launch(EngineArgs a, void* ws, size_t ws_bytes, cudaStream_t stream);
obc_status blocked_engine_launch(EngineArgs a, void* ws, size_t ws_bytes, cudaStream_t stream);

obc_status streaming_engine_plan(int d, int32_t* plan);
obc_status blocked_engine_plan(int d, int with_trace, int row_count, const EngineOpts& eo, int32_t* plan);


}  // namespace obc
