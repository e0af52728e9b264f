// Row elimination engine: Algorithm 1 (ExactOBS pruning) and Algorithm 3 (OBQ) of "Optimal Brain
// Compression", one thread block per weight-matrix row, many rows per launch.
//
// Each row owns a private FP32 copy of the inverse Hessian.  Because the copy stays symmetric under the
// Lemma-1 update, only its lower triangle is stored and updated.  The remaining set M is kept as a
// *leading block*: after slot p is eliminated, the last active slot is moved into slot p, so the update
// of step t touches a dense m x m triangle (m = |M|) and the bytes moved shrink with the problem.
// perm[slot] maps back to original column indices (used for tie-breaks and every output).
//
// The O(m) selection state -- the current weights and the diagonal of the inverse -- is carried in FP64
// in shared memory: the increments that reach it are small (the eliminated weight is the cheapest one),
// so FP32 rounding of the matrix enters the scores only through those small increments.
//
// Per step:  argmin over slots (block reduction)  ->  gather pivot vector v (row part contiguous, column
// part strided) and the last active row  ->  update w, diag, u = v/dpp; move slot `last` into slot p
// ->  stream the triangle once:  H[i][j] -= v[i]*u[j]  (128-bit loads/stores, one warp per matrix row).
// Once m*m fits in shared memory the triangle is moved on chip and the row finishes there.
#include "engine.cuh"

namespace obc {

constexpr int ENGINE_THREADS = 1024;
constexpr int ENGINE_WARPS = ENGINE_THREADS / 32;
constexpr int ENGINE_FIXED_SMEM = 1280;       // 1024 B reduction scratch + broadcast block

struct State {                            // views into shared memory (layout differs per phase)
    double* wd; double* dg; int* perm; float* v; float* u; float* lr;
};

// Block-wide argmin of (score, original index) over slots [0, m).  quant: score uses q(w)-w.
// With outliers: any slot with |q(w)-w| > sc/2 wins by largest error (Section 4, "Quantization Outliers").
__device__ void block_argmin(const State& st, int m, bool quant, bool outliers, Bcast* bc, char* scratch) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double bs = CUDART_INF, oe = -1.0;
    int bo = 0x7fffffff, bslot = -1, oo = 0x7fffffff, oslot = -1;
    const double sc = bc->sc, ze = bc->ze, mq = bc->mq;
    for (int j = tid; j < m; j += ENGINE_THREADS) {
        const double w = st.wd[j];
        double err = -w, code;
        if (quant) err = grid_q(w, sc, ze, mq, &code) - w;
        const double s = err * err / st.dg[j];
        const int o = st.perm[j];
        if (key_less(s, o, bs, bo)) { bs = s; bo = o; bslot = j; }
        if (outliers) {
            const double a = fabs(err);
            if (a > 0.5 * sc && (a > oe || (a == oe && o < oo))) { oe = a; oo = o; oslot = j; }
        }
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) {
        const double s2 = __shfl_xor_sync(0xffffffffu, bs, off);
        const int o2 = __shfl_xor_sync(0xffffffffu, bo, off);
        const int l2 = __shfl_xor_sync(0xffffffffu, bslot, off);
        if (key_less(s2, o2, bs, bo)) { bs = s2; bo = o2; bslot = l2; }
        if (outliers) {
            const double e2 = __shfl_xor_sync(0xffffffffu, oe, off);
            const int p2 = __shfl_xor_sync(0xffffffffu, oo, off);
            const int q2 = __shfl_xor_sync(0xffffffffu, oslot, off);
            if (e2 > oe || (e2 == oe && p2 < oo)) { oe = e2; oo = p2; oslot = q2; }
        }
    }
    double* rs = reinterpret_cast<double*>(scratch);            // [32] scores
    double* re = rs + 32;                                       // [32] outlier errors
    int* ro = reinterpret_cast<int*>(re + 32);                  // [32] orig, [32] slot, [32] o-orig, [32] o-slot
    if (lane == 0) {
        rs[warp] = bs; ro[warp] = bo; ro[32 + warp] = bslot;
        re[warp] = oe; ro[64 + warp] = oo; ro[96 + warp] = oslot;
    }
    __syncthreads();
    if (warp == 0) {
        bs = rs[lane]; bo = ro[lane]; bslot = ro[32 + lane];
        oe = re[lane]; oo = ro[64 + lane]; oslot = ro[96 + lane];
#pragma unroll
        for (int off = 16; off; off >>= 1) {
            const double s2 = __shfl_xor_sync(0xffffffffu, bs, off);
            const int o2 = __shfl_xor_sync(0xffffffffu, bo, off);
            const int l2 = __shfl_xor_sync(0xffffffffu, bslot, off);
            if (key_less(s2, o2, bs, bo)) { bs = s2; bo = o2; bslot = l2; }
            const double e2 = __shfl_xor_sync(0xffffffffu, oe, off);
            const int p2 = __shfl_xor_sync(0xffffffffu, oo, off);
            const int q2 = __shfl_xor_sync(0xffffffffu, oslot, off);
            if (e2 > oe || (e2 == oe && p2 < oo)) { oe = e2; oo = p2; oslot = q2; }
        }
        if (lane == 0) bc->slot = (outliers && oslot >= 0) ? oslot : bslot;
    }
    __syncthreads();
}

// One pass of the Lemma-1 update over the lower triangle held in global memory, in the coordinates that
// hold AFTER slot `last` has been moved into slot pm (pm < 0: nothing moved).  mp = number of rows left.
//   H[i][j] <- base(i,j) - v[i]*u[j],   base = lr[j] on row pm, lr[i] on column pm, else the old H[i][j].
__device__ __forceinline__ void pass_global(float* __restrict__ Hi, int ld, int mp, int pm, const State& st) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float4* u4 = reinterpret_cast<const float4*>(st.u);
    const float4* l4 = reinterpret_cast<const float4*>(st.lr);
    const int pm4 = pm >> 2, pmc = pm & 3;
    const float upm = pm >= 0 ? st.u[pm] : 0.f;
    for (int i = warp; i < mp; i += ENGINE_WARPS) {
        float4* row = reinterpret_cast<float4*>(Hi + (size_t)i * ld);
        const int n4 = (i >> 2) + 1;
        const float nv = -st.v[i];
        {   // The row this warp takes next is pulled into L2 meanwhile (a warp has 2 KB in flight otherwise).  Only
            // rows up to 6 KB: with all SMs one row ahead, longer rows overflow the share of L2 they get and are
            // fetched twice (measured at d_col = 3072: 30 % more DRAM reads, no gain).
            const int inext = i + ENGINE_WARPS;
            if (inext < mp && inext < 1536) {
                const char* nr = reinterpret_cast<const char*>(Hi + (size_t)inext * ld);
                const int bytes = ((inext >> 2) + 1) * 16;
                for (int off = lane * 128; off < bytes; off += 32 * 128)
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(nr + off));
            }
        }
        if (i == pm) {
            for (int j4 = lane; j4 < n4; j4 += 32) {
                const float4 b = l4[j4], u = u4[j4];
                row[j4] = make_float4(fmaf(nv, u.x, b.x), fmaf(nv, u.y, b.y), fmaf(nv, u.z, b.z), fmaf(nv, u.w, b.w));
            }
            continue;
        }
        const bool fix = pm >= 0 && i > pm;
        const float fixval = fix ? fmaf(nv, upm, st.lr[i]) : 0.f;
        for (int j0 = lane; j0 < n4; j0 += 128) {
            float4 a[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int j4 = j0 + 32 * k;
                if (j4 < n4) a[k] = row[j4];
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int j4 = j0 + 32 * k;
                if (j4 < n4) {
                    const float4 u = u4[j4];
                    float4 r = make_float4(fmaf(nv, u.x, a[k].x), fmaf(nv, u.y, a[k].y),
                                           fmaf(nv, u.z, a[k].z), fmaf(nv, u.w, a[k].w));
                    if (fix && j4 == pm4) {
                        if (pmc == 0) r.x = fixval; else if (pmc == 1) r.y = fixval;
                        else if (pmc == 2) r.z = fixval; else r.w = fixval;
                    }
                    row[j4] = r;
                }
            }
        }
    }
}

// Same update on the shared-memory triangle S (leading dimension lds, odd).
__device__ __forceinline__ void pass_shared(float* S, int lds, int mp, int pm, const State& st) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = warp; i < mp; i += ENGINE_WARPS) {
        float* row = S + i * lds;
        const float nv = -st.v[i];
        for (int j = lane; j <= i; j += 32) {
            const float base = (i == pm) ? st.lr[j] : (j == pm ? st.lr[i] : row[j]);
            row[j] = fmaf(nv, st.u[j], base);
        }
    }
}

__global__ void __launch_bounds__(ENGINE_THREADS, 1) row_engine_kernel(const EngineArgs a) {
    extern __shared__ __align__(16) char smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d = a.d, cap = a.cap, ms = a.ms;
    char* scratch = smem;                                       // 1024 B of reduction scratch
    Bcast* bc = reinterpret_cast<Bcast*>(smem + 1024);
    float* wfull = reinterpret_cast<float*>(smem + ENGINE_FIXED_SMEM);   // [cap], original-index weights
    char* regionB = smem + ENGINE_FIXED_SMEM + (size_t)cap * 4;
    float* Hp = a.Hws ? a.Hws + (size_t)blockIdx.x * d * a.ldp : nullptr;
    const int lds = ms + 1;

    for (int rr = blockIdx.x; rr < a.row_count; rr += gridDim.x) {
        const int r = a.row_begin + rr;
        State st;
        st.wd = reinterpret_cast<double*>(regionB);
        st.dg = st.wd + cap;
        st.perm = reinterpret_cast<int*>(st.dg + cap);
        st.v = reinterpret_cast<float*>(st.perm + cap);
        st.u = st.v + cap;
        st.lr = st.u + cap;
        float* S = nullptr;

        int n_forced = 0, n_free = 0;
        bool quant = false;
        if (a.mode == MODE_PRUNE) { n_free = a.steps; }
        else if (a.mode == MODE_REPLAY) { n_forced = a.forced_counts[r]; }
        else if (a.mode == MODE_QUANT) { n_free = d; quant = true; }
        else { n_forced = a.forced_counts[r]; n_free = d - n_forced; quant = true; }
        if (n_forced < 0) n_forced = 0;
        if (n_forced > d) n_forced = d;
        if (n_free > d - n_forced) n_free = d - n_forced;
        const int total = n_forced + n_free;
        const bool outliers = quant && (a.flags & OBC_FLAG_OUTLIERS);

        // ---- row set-up ------------------------------------------------------------------------------
        for (int j = tid; j < d; j += ENGINE_THREADS) {
            const float w = a.W[(size_t)r * a.ldw + j];
            st.wd[j] = (double)w;
            st.dg[j] = (double)a.Hinv[(size_t)j * a.ldhi + j];
            st.perm[j] = j;
            wfull[j] = w;
            if (a.codes) a.codes[(size_t)r * d + j] = -1;
        }
        if (tid == 0) {
            bc->fail = 0;
            bc->sc = 1.0; bc->ze = 0.0; bc->mq = 0.0;
            if (a.mode == MODE_QUANT) {
                bc->sc = (double)a.scale[r]; bc->ze = (double)a.zero[r];
                bc->mq = (double)grid_maxq(a.bits, a.symmetric);
            }
            a.row_status[r] = 0;
        }
        if (a.w_trace)
            for (int j = tid; j < d; j += ENGINE_THREADS)
                a.w_trace[((size_t)r * (a.trace_steps + 1)) * d + j] = a.W[(size_t)r * a.ldw + j];
        bool tail = false;
        const float* src = a.Hinv; int src_ld = a.ldhi;
        if (d > ms && total > 0) {
            // private lower triangle in global memory
            for (int i = warp; i < d; i += ENGINE_WARPS) {
                const float4* s4 = reinterpret_cast<const float4*>(a.Hinv + (size_t)i * a.ldhi);
                float4* d4 = reinterpret_cast<float4*>(Hp + (size_t)i * a.ldp);
                const int n4 = (i >> 2) + 1;
                for (int j0 = lane; j0 < n4; j0 += 128) {      // four loads in flight per lane
                    float4 t[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) if (j0 + 32 * k < n4) t[k] = __ldg(s4 + j0 + 32 * k);
#pragma unroll
                    for (int k = 0; k < 4; ++k) if (j0 + 32 * k < n4) d4[j0 + 32 * k] = t[k];
                }
            }
            src = Hp; src_ld = a.ldp;
        }
        __syncthreads();

        int m = d;
        int s = 0;
        for (; s < total; ++s) {
            // ---- move on chip once the triangle fits ---------------------------------------------------
            if (!tail && m <= ms) {
                double rwd = 0, rdg = 0; int rperm = 0;
                if (tid < m) { rwd = st.wd[tid]; rdg = st.dg[tid]; rperm = st.perm[tid]; }
                __syncthreads();
                st.dg = st.wd + ms;
                st.perm = reinterpret_cast<int*>(st.dg + ms);
                st.v = reinterpret_cast<float*>(st.perm + ms);
                st.u = st.v + ms;
                st.lr = st.u + ms;
                S = st.lr + ms;
                if (tid < m) { st.wd[tid] = rwd; st.dg[tid] = rdg; st.perm[tid] = rperm; }
                for (int i = warp; i < m; i += ENGINE_WARPS)
                    for (int j = lane; j <= i; j += 32) S[i * lds + j] = src[(size_t)i * src_ld + j];
                tail = true;
                __syncthreads();
            }
            const bool forced = s < n_forced;
            const bool q_now = quant && !forced;
            // ---- grid of the compound path: built from the survivors when the replay is over -----------
            if (a.mode == MODE_REPLAY_QUANT && s == n_forced) {
                float lo = 0.f, hi = 0.f;
                for (int j = tid; j < m; j += ENGINE_THREADS) { const float w = (float)st.wd[j]; lo = fminf(lo, w); hi = fmaxf(hi, w); }
#pragma unroll
                for (int off = 16; off; off >>= 1) {
                    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
                    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
                }
                float* rf = reinterpret_cast<float*>(scratch);
                if (lane == 0) { rf[warp] = lo; rf[32 + warp] = hi; }
                __syncthreads();
                if (tid == 0) {
                    for (int k = 0; k < ENGINE_WARPS; ++k) { lo = fminf(lo, rf[k]); hi = fmaxf(hi, rf[32 + k]); }
                    float sc, ze;
                    grid_from_range(lo, hi, a.bits, a.symmetric, &sc, &ze);
                    a.scale[r] = sc; a.zero[r] = ze;
                    bc->sc = (double)sc; bc->ze = (double)ze; bc->mq = (double)grid_maxq(a.bits, a.symmetric);
                }
                __syncthreads();
            }
            // ---- pick the slot -------------------------------------------------------------------------
            if (forced) {
                if (tid == 0) bc->slot = -1;
                __syncthreads();
                const int f = a.forced_order[(size_t)r * d + s];
                for (int j = tid; j < m; j += ENGINE_THREADS)
                    if (st.perm[j] == f) bc->slot = j;
                __syncthreads();
            } else {
                block_argmin(st, m, q_now, outliers, bc, scratch);
            }
            const int p = bc->slot;
            const int last = m - 1;
            if (tid == 0) {
                int fail = 0;
                double dpp = 0, e = 0, qp = 0, code = -1;
                if (p < 0) fail = 1;
                else {
                    bc->op = st.perm[p];
                    dpp = st.dg[p];
                    if (!(dpp > 0.0) || !isfinite(dpp) || !isfinite(st.wd[p])) fail = 1;
                    else {
                        if (q_now) qp = grid_q(st.wd[p], bc->sc, bc->ze, bc->mq, &code);
                        e = st.wd[p] - qp;
                    }
                }
                bc->fail = fail; bc->dpp = dpp; bc->e = e; bc->qp = qp; bc->code = code;
            }
            // ---- pivot vector and last active row --------------------------------------------------------
            if (p >= 0) {
                if (!tail) {
                    const float* rowp = Hp + (size_t)p * a.ldp;
                    for (int j = tid; j <= p; j += ENGINE_THREADS) st.v[j] = rowp[j];
                    for (int i = p + 1 + tid; i < m; i += ENGINE_THREADS) st.v[i] = Hp[(size_t)i * a.ldp + p];
                    const float* rowl = Hp + (size_t)last * a.ldp;
                    for (int j = tid; j <= last; j += ENGINE_THREADS) st.lr[j] = rowl[j];
                } else {
                    for (int j = tid; j < m; j += ENGINE_THREADS) {
                        st.v[j] = (j <= p) ? S[p * lds + j] : S[j * lds + p];
                        st.lr[j] = S[last * lds + j];
                    }
                }
            }
            __syncthreads();
            if (bc->fail) break;
            // ---- O(m) state update (Eq. 3 / Eq. 7), fused with the move of slot `last` into slot p ------
            {
                const double dpp = bc->dpp, f = bc->e / dpp;
                const int op = bc->op;
                for (int j = tid; j < m; j += ENGINE_THREADS) {
                    if (j == p) continue;
                    const float vj = st.v[j];
                    const double nw = st.wd[j] - f * (double)vj;
                    const double nd = st.dg[j] - (double)vj * (double)vj / dpp;
                    const float uj = (float)((double)vj / dpp);
                    const int oj = st.perm[j];
                    wfull[oj] = (float)nw;
                    const int dst = (j == last) ? p : j;       // p != last here
                    st.wd[dst] = nw; st.dg[dst] = nd; st.u[dst] = uj;
                    if (j == last) { st.perm[p] = oj; st.v[p] = vj; st.lr[p] = st.lr[last]; }
                }
                if (tid == 0) {
                    wfull[op] = (float)bc->qp;
                    if (!forced) {
                        const int t = s - n_forced;
                        if (a.order) a.order[(size_t)r * d + t] = op;
                        if (a.loss) a.loss[(size_t)r * d + t] = (float)(bc->e * bc->e / dpp);
                    }
                    if (q_now && a.codes) a.codes[(size_t)r * d + op] = (int)bc->code;
                }
            }
            __syncthreads();
            if (a.w_trace && s < a.trace_steps)
                for (int j = tid; j < d; j += ENGINE_THREADS)
                    a.w_trace[((size_t)r * (a.trace_steps + 1) + s + 1) * d + j] = wfull[j];
            // ---- Lemma 1 on the triangle ------------------------------------------------------------------
            const int pm = (p == last) ? -1 : p;
            if (s + 1 < total) {
                if (!tail) pass_global(Hp, a.ldp, m - 1, pm, st);
                else pass_shared(S, lds, m - 1, pm, st);
            }
            --m;
            __syncthreads();
        }
        // ---- row epilogue ---------------------------------------------------------------------------------
        if (s < total) {        // stopped early: report the step, mark what was not produced
            if (tid == 0) a.row_status[r] = 1 + s;
            const int t0 = (s < n_forced) ? 0 : s - n_forced;
            for (int t = t0 + tid; t < n_free; t += ENGINE_THREADS) {
                if (a.order) a.order[(size_t)r * d + t] = -1;
                if (a.loss) a.loss[(size_t)r * d + t] = CUDART_INF_F;
            }
        }
        if (a.W_out)
            for (int j = tid; j < d; j += ENGINE_THREADS) a.W_out[(size_t)r * a.ldwo + j] = wfull[j];
        __syncthreads();
    }
}

// ---- host side ---------------------------------------------------------------------------------------------
static size_t engine_smem_bytes(int cap, int ms) {
    const size_t phase1 = (size_t)36 * cap;
    const size_t tailb = (size_t)36 * ms + (size_t)4 * ms * (ms + 1);
    return ENGINE_FIXED_SMEM + (size_t)4 * cap + (phase1 > tailb ? phase1 : tailb);
}

// Largest even on-chip threshold that fits the opt-in shared memory next to the per-row state.
static int engine_pick_ms(int d, int cap, int smem_optin) {
    int ms = d < 1024 ? d : 1024;
    ms &= ~1;
    if (ms < 2) ms = 2;
    while (ms > 2 && engine_smem_bytes(cap, ms) > (size_t)smem_optin) ms -= 2;
    return ms;
}

size_t streaming_engine_workspace_bytes(int row_count, int d, const DeviceInfo& di) {
    const int cap = (d + 3) & ~3;
    const int ms = engine_pick_ms(d, cap, di.smem_optin);
    if (d <= ms) return 256;
    int blocks = di.sm_count;
    if (row_count > 0 && row_count < blocks) blocks = row_count;
    return round_up((size_t)blocks * d * cap * sizeof(float), 256);
}

obc_status streaming_engine_launch(EngineArgs a, void* ws, size_t ws_bytes, cudaStream_t stream) {
    DeviceInfo di;
    obc_status st = device_info(&di);
    if (st != OBC_OK) return st;
    a.cap = (a.d + 3) & ~3;
    if (a.d > OBC_MAX_DCOL || engine_smem_bytes(a.cap, 2) > (size_t)di.smem_optin) return OBC_ERR_UNSUPPORTED;
    a.ms = engine_pick_ms(a.d, a.cap, di.smem_optin);
    int blocks = di.sm_count < a.row_count ? di.sm_count : a.row_count;
    const size_t need = streaming_engine_workspace_bytes(a.row_count, a.d, di);
    if (!ws || !aligned256(ws) || ws_bytes < need) return OBC_ERR_WORKSPACE;
    a.Hws = reinterpret_cast<float*>(ws);
    a.ldp = a.cap;
    const size_t smem = engine_smem_bytes(a.cap, a.ms);
    OBC_CUDA_TRY(cudaFuncSetAttribute(row_engine_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    row_engine_kernel<<<blocks, ENGINE_THREADS, smem, stream>>>(a);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

obc_status streaming_engine_plan(int d, int32_t* plan) {
    DeviceInfo di;
    obc_status st = device_info(&di);
    if (st != OBC_OK) return st;
    const int cap = (d + 3) & ~3;
    if (d > OBC_MAX_DCOL || engine_smem_bytes(cap, 2) > (size_t)di.smem_optin) return OBC_ERR_UNSUPPORTED;
    plan[0] = OBC_ENGINE_STREAMING; plan[1] = ENGINE_THREADS; plan[2] = 1; plan[3] = engine_pick_ms(d, cap, di.smem_optin);
    plan[4] = 0; plan[5] = 1; plan[6] = di.sm_count; plan[7] = 0;
    return OBC_OK;
}

// ---- engine choice ----------------------------------------------------------------------------------------
size_t engine_workspace_bytes(int row_count, int d, const DeviceInfo& di) {
    const size_t s1 = streaming_engine_workspace_bytes(row_count, d, di);
    const size_t s2 = blocked_engine_workspace_bytes(row_count, d, di);
    return s1 > s2 ? s1 : s2;          // valid for either engine, whichever is selected at call time
}

static obc_status engine_launch(EngineArgs a, void* ws, size_t ws_bytes, cudaStream_t stream) {
    if (a.opts.engine == OBC_ENGINE_STREAMING) return streaming_engine_launch(a, ws, ws_bytes, stream);
    return blocked_engine_launch(a, ws, ws_bytes, stream);
}

static EngineArgs base_args(const float* W, int ldw, int d_col, int row_begin, int row_count, const float* Hinv,
                            int ldhi, int32_t* row_status, const EngineOpts& eo) {
    EngineArgs a = {};
    a.opts = eo;
    a.W = W; a.ldw = ldw; a.d = d_col; a.row_begin = row_begin; a.row_count = row_count;
    a.Hinv = Hinv; a.ldhi = ldhi; a.row_status = row_status;
    a.bits = 2;
    return a;
}

obc_status engine_prune_trace(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                              const float* Hinv, int ldhi, int steps, int32_t* order, float* loss, float* w_trace,
                              int32_t* row_status, void* ws, size_t ws_bytes, const EngineOpts& eo, cudaStream_t stream) {
    (void)d_row;
    EngineArgs a = base_args(W, ldw, d_col, row_begin, row_count, Hinv, ldhi, row_status, eo);
    a.mode = MODE_PRUNE; a.steps = steps; a.order = order; a.loss = loss;
    a.w_trace = w_trace; a.trace_steps = steps;
    return engine_launch(a, ws, ws_bytes, stream);
}

obc_status engine_prune_nm(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                           const float* Hinv, int ldhi, int n_keep, int m_block, int32_t* order, float* loss,
                           float* W_out, int ldwo, uint8_t* mask, int32_t* row_status, void* ws, size_t ws_bytes,
                           const EngineOpts& eo, cudaStream_t stream) {
    (void)d_row;
    EngineArgs a = base_args(W, ldw, d_col, row_begin, row_count, Hinv, ldhi, row_status, eo);
    a.mode = MODE_PRUNE; a.steps = d_col / m_block * (m_block - n_keep); a.order = order; a.loss = loss;
    a.trace_steps = a.steps; a.W_out = W_out; a.ldwo = ldwo; a.mask = mask;
    a.nm_prune = m_block - n_keep;
    a.nm_lg = 0;
    while ((1 << a.nm_lg) < m_block) ++a.nm_lg;
    return blocked_engine_launch(a, ws, ws_bytes, stream);      // the pattern is built into the blocked engine only
}

obc_status engine_prune_blocks(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                               const float* Hinv, int ldhi, int block, int32_t* order, float* loss, float* w_trace,
                               int32_t* row_status, void* ws, size_t ws_bytes, const EngineOpts& eo, cudaStream_t stream) {
    (void)d_row;
    EngineArgs a = base_args(W, ldw, d_col, row_begin, row_count, Hinv, ldhi, row_status, eo);
    a.mode = MODE_PRUNE; a.steps = d_col; a.order = order; a.loss = loss; a.w_trace = w_trace; a.trace_steps = d_col;
    a.block_c = block;
    return blocked_engine_launch(a, ws, ws_bytes, stream);
}

// Block pruning keeps every row in global memory to the end (no on-chip tail), so it needs the private triangles
// at any row length.
size_t engine_blocks_workspace_bytes(int row_count, int d, const DeviceInfo& di) {
    const int cap = (d + 3) & ~3;
    int blocks = di.sm_count * 4;
    if (row_count > 0 && row_count < blocks) blocks = row_count;
    const size_t tri = round_up((size_t)blocks * d * cap * sizeof(float), 256);
    const size_t other = blocked_engine_workspace_bytes(row_count, d, di);
    return tri > other ? tri + 256 : other;
}

obc_status engine_replay(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                         const float* Hinv, int ldhi, const int32_t* order, const int32_t* counts, float* W_out,
                         int ldwo, int32_t* row_status, void* ws, size_t ws_bytes, const EngineOpts& eo, cudaStream_t stream) {
    (void)d_row;
    EngineArgs a = base_args(W, ldw, d_col, row_begin, row_count, Hinv, ldhi, row_status, eo);
    a.mode = MODE_REPLAY; a.forced_order = order; a.forced_counts = counts; a.W_out = W_out; a.ldwo = ldwo;
    return engine_launch(a, ws, ws_bytes, stream);
}

obc_status engine_quantize(const float* W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                           const float* Hinv, int ldhi, float* scale, float* zero, int bits, int symmetric,
                           const int32_t* prune_order, const int32_t* prune_counts, int flags, float* W_out,
                           int ldwo, int32_t* codes, float* loss, int32_t* qorder, int32_t* row_status, void* ws,
                           size_t ws_bytes, const EngineOpts& eo, cudaStream_t stream) {
    (void)d_row;
    EngineArgs a = base_args(W, ldw, d_col, row_begin, row_count, Hinv, ldhi, row_status, eo);
    a.mode = prune_order ? MODE_REPLAY_QUANT : MODE_QUANT;
    a.forced_order = prune_order; a.forced_counts = prune_counts;
    a.scale = scale; a.zero = zero; a.bits = bits; a.symmetric = symmetric; a.flags = flags;
    a.W_out = W_out; a.ldwo = ldwo; a.codes = codes; a.loss = loss; a.order = qorder;
    return engine_launch(a, ws, ws_bytes, stream);
}

}  // namespace obc
