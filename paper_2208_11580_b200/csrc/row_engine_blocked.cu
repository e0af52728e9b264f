// Row elimination engine with deferred Lemma-1 updates (Algorithm 1 / Algorithm 3 of "Optimal Brain
// Compression"), one thread block per weight-matrix row, several rows per SM.
//
// A greedy step needs only three things from the row's inverse Hessian: its diagonal (for the scores), the
// pivot column (for the weight update, Eq. 3 / Eq. 7) and, later, everything else.  Lemma 1 is a rank-1
// update, so B of them can be held back as vectors z_b = H[:,p_b] / sqrt([H]_pp) (each taken from the matrix
// as it would be at its own step) and applied together:
//       H_true = H_stored - sum_b z_b z_b^T .
// The pivot column of a step is then one column of H_stored corrected by the pending vectors (m x B work),
// and the m x m matrix is read and written once per B steps instead of once per step.  Picks, weights and
// losses are the same as with step-by-step updates up to the order of the FP32 roundings.
//
// Layout.  The private copy keeps the lower triangle only (the matrix stays symmetric).  Slots [0, m0) are
// fixed between two flushes; eliminated slots are marked dead (perm = -1).  The flush applies the pending
// vectors and compacts at the same time: a dead slot h below the new size m1 is taken over by a live slot
// s >= m1, i.e. element (i, j) of the new triangle is read from (max(si, sj), min(si, sj)) of the old one.
// All such foreign reads come from rows >= m1, which the flush never writes, so it runs in place.
// The flush is a rank-B update and runs on the tensor cores (warp tiles of 16 rows x 64 columns, TF32 split
// products, see blk_flush_mma); the pending vectors stay in shared memory (at very long rows further ones sit in a
// global buffer that stays in L2; the flush reads their operands from there).  The O(m) selection state (weights, diagonal) is FP64, as in
// the streaming engine.  Once the live triangle fits into the shared memory of the pending vectors, the row
// finishes on chip with step-by-step updates.
//
// Shares of rows.  When a launch has more rows than resident blocks and the rows do not divide evenly, whole waves
// would leave most SMs idle through the last one.  Instead every block gets the same amount of work: the rows
// are laid end to end and cut into gridDim.x equal pieces.  A row that straddles a cut is started by the block before
// the cut -- as that block's FIRST item -- up to a flush boundary near the cut, where its state (weights, diagonal,
// slot map; the triangle stays in a buffer of its own) is saved, and it is finished by the next block as that
// block's LAST item.  The state is complete long before it is needed; the reader still checks a flag with a bounded
// wait (a cooperative launch keeps all blocks resident) and reports a row it could not pick up through row_status.
//
// Step protocol.  Between two flushes every slot belongs to one thread (groups of 4 consecutive slots per
// thread), which is the only one to touch wd[j], dg[j], perm[j] and its entries of the pending vectors; the
// update phase also leaves an FP32 estimate of each own slot's next score in registers.  Each thread proposes its best slot, the
// warps combine the proposals and publish one record per warp (with the candidate's weight and diagonal),
// and after the single barrier of the step every warp reads the records and derives the same winner, so
// no second barrier is needed to announce it.  Records alternate between two buffers by step parity.
#include "engine.cuh"

namespace obc {

constexpr int BLK_MAXB = 64;
constexpr int BLK_REC_BYTES = 640;            // one record buffer: 16 warps x (key, slot, orig, s, w, dg)
constexpr int BLK_OFF_BC = 1280;              // Bcast (grid parameters, flush bookkeeping)
constexpr int BLK_OFF_PV = 1536;              // int pv[64]   slots eliminated since the last flush
constexpr int BLK_OFF_HL = 1792;              // int hl[64]   holes (dead slots below the new size)
constexpr int BLK_OFF_MV = 2048;              // int mv[64]   live slots that move into the holes
constexpr int BLK_OFF_CM = 2304;
constexpr int BLK_OFF_RF = 2944;              // float rf[64]  min/max reduction of the compound grid
constexpr int BLK_OFF_GRP = 3200;             // forced groups: int slot[4], float M[4][4] (pivot columns at the pivot slots)
constexpr int BLK_OFF_SCHED = 3280;           // int[12]: kind of the item in work (shares of rows)
constexpr int BLK_FIXED = 3328;
constexpr int BLK_GS = 4;                     // forced eliminations taken together

// Per-row state in shared memory: wd, dg (FP64), perm (int32), srcm (uint16); optional: the row in original
// order (weight trace), one byte per block of the N:M pattern.
// (block pruning, bc = block size 4 or 8: the 6 or 28 off-diagonal entries of every block's c x c diagonal block, FP64)
__host__ __device__ inline size_t blk_state_bytes(int cap, bool wfull, bool nm = false, int bc = 0) {
    return (size_t)20 * cap + (((size_t)2 * cap + 15) & ~(size_t)15) + (wfull ? (size_t)4 * cap : 0) +
           (nm ? (((size_t)(cap >> 1) + 15) & ~(size_t)15) : 0) + (bc == 8 ? (size_t)28 * cap : (bc ? (size_t)12 * cap : 0));
}
// Stride of the pending vectors for a row of m slots: = 8 (mod 32), so that the tensor-core fragments of the
// flush (4 vectors x 8 consecutive slots per load) touch 32 different banks.
__host__ __device__ inline int blk_ldz(int m) { return ((m + 8 + 31) & ~31) + 8; }     // >= m + 16
static size_t blk_tail_bytes(int ms) { return (size_t)12 * ((ms + 3) & ~3) + (size_t)4 * ms * (ms + 1); }

// ---- shares of rows ------------------------------------------------------------------------------------------------
constexpr int BLK_SPLIT_WAIT_LIMIT = 1 << 22;  // polls (256 ns apart) before a block gives up on a row its neighbour started
struct SplitHeader {                          // what the block that started a row leaves for the one that finishes it
    int s_cut;                                // steps done (0: the row was not started)
    int m0;                                   // live slots, all in [0, m0), nothing pending
    int done;                                 // 1: nothing is left to do (the row was finished, or failed and was reported)
    int pad[61];
};
// followed by: double wd[cap], double dg[cap], int perm[cap], float wfull[cap]
__host__ __device__ inline size_t blk_split_stride(int cap) { return sizeof(SplitHeader) + (size_t)28 * cap + 256; }

// Work model of a row, in units of "half a matrix element moved by a flush": a pass over the compacted triangle of m
// slots costs m^2 / 2, a deferred-update step costs as much as BLK_STEP_COST of those (measured on B200: a pass takes
// 1.1 - 1.3e-10 s per m^2; a step 7 us with one 512-thread row per SM, 3.4 us with several smaller blocks per SM).
__host__ __device__ inline double blk_step_cost(int nt) { return nt >= 512 ? 30000.0 : 14000.0; }

// The flush boundary of a row's schedule at which about num/den of the row's work is done (0: before the first
// boundary; total: the share reaches into the on-chip end of the row, which is then left to the starting block).
// Every thread of a block computes the same value from the same arguments.
__device__ __noinline__ int blk_cut_step(int d, int ms, int total, int panel_floats, int max_pending, int g_vectors,
                                        int num, int den, double step_cost) {
    double all = 0.0, at = 0.0;
    int cut = 0;
    for (int pass = 0; pass < 2; ++pass) {
        int m = d, s = 0;
        double cost = 0.0;
        while (s < total && m > ms) {
            int b = min(max_pending, panel_floats / blk_ldz(m) + g_vectors);
            b = max(1, min(b, min(m - ms, total - s)));
            cost += step_cost * b;
            s += b; m -= b;
            if (s >= total) break;
            cost += 0.5 * (double)m * (double)m;                  // the pass over the compacted triangle
            if (pass == 1 && m > ms && cost <= at) cut = s;       // last boundary not beyond the share
        }
        cost += step_cost * 0.6 * (total - s);                    // steps on chip
        if (pass == 0) { all = cost; at = all * (double)num / (double)den; }
    }
    return cut;
}

// The it-th item of block `blk` out of `ng` when `rows` rows are shared out: false when there is none.  Without
// shares: whole rows blk, blk + ng, ...  With shares: positions in units of 1/ng of a row, row r covers
// [r ng, (r+1) ng) and the block covers [blk rows, (blk+1) rows); the row that straddles the upper cut is started first
// (head_num/ng of it), the one that straddles the lower cut is finished last.  Plain integer arithmetic, recomputed
// per item so that nothing of it stays in registers during a row.
enum { ITEM_FULL = 0, ITEM_HEAD = 1, ITEM_TAIL = 2 };
__device__ __forceinline__ bool blk_item(bool split, int blk, int ng, int rows, int it, int* rr, int* kind, int* head_num) {
    *kind = ITEM_FULL; *head_num = 0;
    if (!split) { *rr = blk + it * ng; return *rr < rows; }
    const long long a0 = (long long)blk * rows, a1 = a0 + rows;
    const int r_first = (int)(a0 / ng), tail_num = (int)(a0 - (long long)r_first * ng);
    const int r_last = (int)((a1 - 1) / ng);
    int hn = (int)(a1 - (long long)r_last * ng);
    if (hn == ng) hn = 0;                                          // the row ends at the cut: a whole row
    const int full_lo = tail_num ? r_first + 1 : r_first, full_hi = hn ? r_last : r_last + 1;
    const int n_items = (hn ? 1 : 0) + (full_hi - full_lo) + (tail_num ? 1 : 0);
    if (it >= n_items) return false;
    if (hn && it == 0) { *rr = r_last; *kind = ITEM_HEAD; *head_num = hn; }
    else if (tail_num && it == n_items - 1) { *rr = r_first; *kind = ITEM_TAIL; }
    else *rr = full_lo + it - (hn ? 1 : 0);
    return true;
}

// The cold paths of the hand-over are kept out of line, so that the register allocation of a row's loop is the
// same with and without them.
// Thread 0: wait (bounded) for the flag of the block that started the row; returns 1 when it is set.
__device__ __noinline__ int blk_wait_flag(int* flag) {
    int ok = 0;
    for (int spin = 0; spin < BLK_SPLIT_WAIT_LIMIT; ++spin) {
        if (atomicAdd(flag, 0) != 0) { ok = 1; break; }
        __nanosleep(256);
    }
    __threadfence();
    return ok;
}
// Thread 0: publish the header of the row this block started (or declined to start), then the flag.
__device__ __noinline__ void blk_publish(char* state, int* flag, int s_cut, int m0, int done) {
    SplitHeader* sh = reinterpret_cast<SplitHeader*>(state);
    sh->s_cut = s_cut; sh->m0 = m0; sh->done = done;
    __threadfence();
    atomicExch(flag, 1);
}
// All threads: state of a row between shared memory and the hand-over record (save = true: to the record).
__device__ __noinline__ void blk_state_copy(bool save, char* state, int cap, int d, int m, int nt, double* wd, double* dg,
                                            int* perm, unsigned short* srcm, float* wfull) {
    char* base = state + sizeof(SplitHeader);
    double* swd = reinterpret_cast<double*>(base);
    double* sdg = swd + cap;
    int* sperm = reinterpret_cast<int*>(sdg + cap);
    float* swf = reinterpret_cast<float*>(sperm + cap);
    const int tid = threadIdx.x;
    if (save) {
        for (int j = tid; j < m; j += nt) { swd[j] = wd[j]; sdg[j] = dg[j]; sperm[j] = perm[j]; }
        if (wfull) for (int j = tid; j < d; j += nt) swf[j] = wfull[j];
        __threadfence();                   // state, triangle and outputs of every thread before the flag
    } else {
        for (int j = tid; j < cap; j += nt) {
            const bool in = j < m;
            wd[j] = in ? swd[j] : 0.0; dg[j] = in ? sdg[j] : 0.0; perm[j] = in ? sperm[j] : -1;
            srcm[j] = (unsigned short)j;
            if (wfull && j < d) wfull[j] = swf[j];
        }
    }
}

struct Records {                              // views into one record buffer
    unsigned* key; int* slot; int* orig; double* s; double* w; double* dgv;
};
__device__ __forceinline__ Records rec_view(char* scratch, int parity) {
    char* b = scratch + parity * BLK_REC_BYTES;
    Records r;
    r.s = reinterpret_cast<double*>(b);       // [16]
    r.w = r.s + 16;                           // [16]
    r.dgv = r.w + 16;                         // [16]
    r.key = reinterpret_cast<unsigned*>(r.dgv + 16);
    r.slot = reinterpret_cast<int*>(r.key + 16);
    r.orig = r.slot + 16;
    return r;
}

// Monotone map of a float to an unsigned key (smaller float -> smaller key); NaN never reaches it.
__device__ __forceinline__ unsigned float_key(float x) {
    const unsigned u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
constexpr unsigned KEY_NONE = 0xFFFFFFFFu;

struct Pick { int slot; int orig; double w; double dgv; double s; };

// Combines one candidate per lane into the lane holding the smallest (s, orig); key = float_key((float)s)
// orders all but near-equal candidates, which are then compared exactly.  Returns the winning lane or -1.
__device__ __forceinline__ int warp_winner(unsigned key, double s, int orig) {
    const unsigned kmin = __reduce_min_sync(0xffffffffu, key);
    if (kmin == KEY_NONE) return -1;
    const unsigned cand = __ballot_sync(0xffffffffu, key == kmin);
    if (__popc(cand) == 1) return __ffs(cand) - 1;
    double bs = (key == kmin) ? s : CUDART_INF;
    int bo = (key == kmin) ? orig : 0x7fffffff;
    int bl = threadIdx.x & 31;
#pragma unroll
    for (int off = 16; off; off >>= 1) {
        const double s2 = __shfl_xor_sync(0xffffffffu, bs, off);
        const int o2 = __shfl_xor_sync(0xffffffffu, bo, off);
        const int l2 = __shfl_xor_sync(0xffffffffu, bl, off);
        if (key_less(s2, o2, bs, bo)) { bs = s2; bo = o2; bl = l2; }
    }
    return bl;
}

// Every thread holds at most one candidate (slot < 0: none).  Publishes the warp's best in the record buffer,
// then, after the barrier, every warp derives the block's best from the records.
template <int NT>
__device__ __forceinline__ Pick block_pick(unsigned key, double s, int slot, int orig, double w, double dgv,
                                           const Records& rec) {
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (slot < 0) key = KEY_NONE;
    const int wl = warp_winner(key, s, orig);
    if (wl < 0) { if (lane == 0) rec.key[warp] = KEY_NONE; }
    else if (lane == wl) {
        rec.key[warp] = key; rec.slot[warp] = slot; rec.orig[warp] = orig;
        rec.s[warp] = s; rec.w[warp] = w; rec.dgv[warp] = dgv;
    }
    __syncthreads();
    const bool in = lane < NW;
    const unsigned k2 = in ? rec.key[lane] : KEY_NONE;
    const double s2 = (in && k2 != KEY_NONE) ? rec.s[lane] : CUDART_INF;
    const int o2 = (in && k2 != KEY_NONE) ? rec.orig[lane] : 0x7fffffff;
    const int ww = warp_winner(k2, s2, o2);
    Pick p;
    p.slot = -1; p.orig = -1; p.w = 0.0; p.dgv = 0.0; p.s = 0.0;
    if (ww >= 0) { p.slot = rec.slot[ww]; p.orig = rec.orig[ww]; p.w = rec.w[ww]; p.dgv = rec.dgv[ww]; p.s = rec.s[ww]; }
    return p;
}

// Slot ownership between two flushes: thread t owns the slots 4t .. 4t+3 of every group of 4 NT slots, i.e.
// slot(k) = (k / 4) * 4 NT + 4 t + (k % 4) for k < KMAX, so that its entries of a pending vector, of a matrix
// row and of the state arrays are 16 contiguous bytes.
template <int NT>
__device__ __forceinline__ int own_slot(int k) { return (k >> 2) * (4 * NT) + (threadIdx.x << 2) + (k & 3); }

// err = q(w) - w on the row's grid.  Kept out of line: it is reached once per slot and step in the OBQ kernels,
// and inlining it at every use multiplies the code size of a kernel whose instruction footprint already matters
// (several rows in different phases share one SM's instruction cache).
__device__ __noinline__ double grid_error(double w, double sc, double isc, double ze, double mq) {
    double code;
    return grid_q_fast(w, sc, isc, ze, mq, &code) - w;
}

// FP32 estimate of the score of a slot (relative error of a few 1e-7): it only screens candidates, the slots
// within 1e-4 of the thread's best estimate are scored again with the FP64 division.
template <bool Q>
__device__ __forceinline__ float score_estimate(double w, double dgv, bool quant, double sc, double isc, double ze,
                                                double mq) {
    if (Q && quant) {
        // plain product and rounding: next to a rounding boundary the two possible codes give the same |err| to
        // ~1e-16, which is all an estimate needs (the exact scoring goes through grid_error)
        const double c = fmin(fmax(rint(w * isc) + ze, 0.0), mq);
        const double err = sc * (c - ze) - w;
        return __fdividef(__double2float_rn(err * err), __double2float_rn(dgv));
    }
    const float wf = __double2float_rn(w);
    return __fdividef(wf * wf, __double2float_rn(dgv));
}

// Estimates of all own slots from the state arrays (NaN for dead or unused slots).
// N:M pattern: blkcnt (nullable) holds per block of 2^nm_lg original columns the number of weights eliminated so
// far; a slot whose block has reached nm_prune is no candidate (NaN estimate).  cntw receives the counts of the
// own slots' blocks, one byte per slot, which the update phase then keeps current in registers.
template <int NT, int KMAX, bool Q>
__device__ __forceinline__ void estimate_own(float (&sa)[KMAX], const double* wd, const double* dg, const int* perm,
                                             int m0, bool quant, double sc, double isc, double ze, double mq,
                                             const unsigned char* blkcnt, int nm_lg, int nm_prune,
                                             unsigned (&cntw)[KMAX / 4]) {
#pragma unroll
    for (int g = 0; g < KMAX / 4; ++g) cntw[g] = 0u;
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
        const int j = own_slot<NT>(k);
        sa[k] = CUDART_NAN_F;
        if (j < m0 && perm[j] >= 0) {
            unsigned c = 0u;
            if (blkcnt) { c = blkcnt[perm[j] >> nm_lg]; cntw[k >> 2] |= c << (8 * (k & 3)); }
            if (!blkcnt || (int)c < nm_prune) sa[k] = score_estimate<Q>(wd[j], dg[j], quant, sc, isc, ze, mq);
        }
    }
}

// The thread's best live slot among its own by (score, original index), given the estimates: only the slots
// within 1e-4 of the thread's best estimate take the FP64 division, so the result (ties included) is the
// exact FP64 choice.  The candidates are first collected in a bit mask and then scored in one loop, so the
// exact scoring exists once in the code and the lanes of a warp take it together.
// With the outlier rule (Section 4, "Quantization Outliers") a slot whose error exceeds Delta/2 wins by
// largest error; such candidates get negative scores, below every regular one.
template <int NT, int KMAX, bool Q>
__device__ __forceinline__ void thread_best(const float (&sa)[KMAX], const double* wd, const double* dg,
                                            const int* perm, bool quant, bool outliers, double sc, double isc,
                                            double ze, double mq, unsigned* key, double* s_out, int* slot_out) {
    float smin = CUDART_INF_F;
#pragma unroll
    for (int k = 0; k < KMAX; ++k) smin = fminf(smin, sa[k]);           // fminf ignores NaN estimates
    const float thr = smin + 1e-4f * fabsf(smin);
    unsigned cand = 0u, valid = 0u;
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
        if (sa[k] <= thr || sa[k] == smin) cand |= 1u << k;             // false for NaN estimates
        if (sa[k] == sa[k]) valid |= 1u << k;
    }
    double bs = CUDART_INF, oe = -1.0;
    int bo = 0x7fffffff, bslot = -1, oo = 0x7fffffff, oslot = -1;
    unsigned todo = (Q && outliers) ? valid : cand;
    while (todo) {
        const int k = __ffs(todo) - 1;
        todo &= todo - 1;
        const int j = own_slot<NT>(k);
        const double w = wd[j];
        double err = -w;
        if (Q && quant) err = grid_error(w, sc, isc, ze, mq);
        const int o = perm[j];
        if ((cand >> k) & 1u) {
            const double s = err * err / dg[j];
            if (key_less(s, o, bs, bo)) { bs = s; bo = o; bslot = j; }
        }
        if (Q && outliers) {
            const double a = fabs(err);
            if (a > 0.5 * sc && (a > oe || (a == oe && o < oo))) { oe = a; oo = o; oslot = j; }
        }
    }
    *key = KEY_NONE; *s_out = bs; *slot_out = bslot;
    if (bslot >= 0) *key = float_key(__double2float_rn(bs));
    if (Q && outliers && oslot >= 0) { *s_out = -oe; *slot_out = oslot; *key = float_key(__double2float_rn(-oe)); }
}

// The flush applies the nb pending vectors Z[b][.] (already in the new slot numbering) to the triangle and compacts it
// to m1 rows.  srcm[i] = old slot whose data new slot i takes (i itself unless i is a hole).  The triangle is far
// larger than L2 and touched once per flush, so it is loaded and stored with the evict-first hint and leaves L2 to
// the overflow part of the pending vectors.
// ---- flush on the tensor cores -----------------------------------------------------------------------------------
// The flush is a rank-nb update, H -= Z^T Z with nb <= 64: a dense contraction.  A warp takes tiles of 16 rows x
// 64 columns; the increment of a tile is formed by mma.sync m16n8k8 (TF32 inputs, FP32 accumulation over 8 pending
// vectors at a time, the partial sums added up in FP32 registers) with every FP32 operand split into two TF32 parts, z = hi + lo, and the three products
// hi*hi + hi*lo + lo*hi (the missing lo*lo term is below 2^-22 of each product, and the products of one update are
// about 1/d_col of the element they change).  The tile of H is fetched afterwards (a prefetch cursor has pulled it
// into L2); the increment is subtracted in FP32 -- one rounding of the matrix element per flush -- and stored.
// Register layout: lane (g, t) = (lane / 4, lane % 4) holds rows g and g + 8 and, of every 16-column group u, the
// four columns 16u + 4t .. + 3 (one 128-bit access per row and group).  The two 8-column MMA tiles of a group take
// its even and its odd columns: tile 2u, n = 2t + e  <->  column 16u + 4t + 2e;  tile 2u+1: that + 1.  Their B
// fragments (n = g) are then the adjacent pair 16u + 2g, + 1 of a pending vector: one 64-bit shared-memory load.
// The leading part is rounded to nearest (on the magnitude, ties away): truncation would leave every product short
// by a part of the same sign, a bias that adds up over the d_col updates of an element instead of averaging out.
__device__ __forceinline__ uint32_t tf32_rn(float x) { return (__float_as_uint(x) + 0x1000u) & 0xFFFFE000u; }
__device__ __forceinline__ void tf32_split(float x, uint32_t& hi, uint32_t& lo) {
    hi = tf32_rn(x);                                        // 11 significant bits
    // the difference is exact in FP32 and has either sign; the tensor core reads its leading 11 bits (truncation of
    // a part whose sign is random is no bias; rounding it too was measured and changes nothing)
    lo = __float_as_uint(x - __uint_as_float(hi));
}
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// GP: pending vectors nbs .. nb - 1 are rows of G (global memory, stride gld: the overflow part, resident in L2).  Their
// row operands are copied once per row group into the warp's staging block zstage (16 floats per vector); their column
// operands are read from L2 in the fragment layout, 8 vectors at a time.
// first product of a chain: the accumulator operand is zero
__device__ __forceinline__ void mma_tf32_z(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}
// two values at once: the integer part of the split per value, the subtraction as one packed FP32 instruction
__device__ __forceinline__ void tf32_split2(float2 x, uint32_t& hi0, uint32_t& hi1, uint32_t& lo0, uint32_t& lo1) {
    hi0 = tf32_rn(x.x); hi1 = tf32_rn(x.y);
    const float2 l = __ffma2_rn(make_float2(__uint_as_float(hi0), __uint_as_float(hi1)), make_float2(-1.f, -1.f), x);
    lo0 = __float_as_uint(l.x); lo1 = __float_as_uint(l.y);
}

template <int NT, bool STREAM, bool GP>
__device__ __forceinline__ void blk_flush_mma(float* __restrict__ Hp, int ldp, int m1, int nb, int nbs, const float* Z, int ldz,
                                              const float* __restrict__ G, int gld, float* zstage,
                                              const unsigned short* srcm, const uint32_t* colmask) {
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int nrg = (m1 + 15) >> 4;
    const int ksteps = ((GP ? nbs : nb) + 7) >> 3;
    const int nbg = GP ? nb - nbs : 0;
    const int ksteps_g = (nbg + 7) >> 3;
    // The products are cheap next to the latency of memory, and a warp has one tile (4 KB) in registers at a time:
    // a cursor runs FLUSH_AHEAD tiles ahead of the warp through its sequence of tiles and pulls them into L2
    // (measured at d_col = 2304: 12 % off the pass with a distance of 1 or 2 tiles, less with 4, a loss from 8 on).
    constexpr int FLUSH_AHEAD = 2;
    int prg = warp, pc0 = 0;
    auto prefetch_next = [&]() {
        if (prg >= nrg) return;
        const int row = (prg << 4) + (lane >> 1), col = pc0 + ((lane & 1) << 5);       // 16 rows x 2 lines of 128 bytes
        if (row < m1 && col <= row)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(Hp + (size_t)srcm[row] * ldp + col));
        pc0 += 64;
        if (pc0 >= min((prg << 4) + 16, m1)) { pc0 = 0; prg += NW; }
    };
#pragma unroll
    for (int a = 0; a < FLUSH_AHEAD; ++a) prefetch_next();
    for (int rg = warp; rg < nrg; rg += NW) {
        const int i0 = rg << 4;
        const int jend = min(i0 + 16, m1);                     // columns [0, jend) hold data of this row group
        const int rr[2] = {i0 + g, i0 + g + 8};                // the lane's two rows
        const bool in[2] = {rr[0] < m1, rr[1] < m1};
        const int sr[2] = {in[0] ? (int)srcm[rr[0]] : 0, in[1] ? (int)srcm[rr[1]] : 0};
        if (GP && nbg > 0) {                                   // row operands of the overflow vectors -> staging block
            __syncwarp();
            for (int e = lane; e < nbg * 4; e += 32) {
                const int v = e >> 2, q = e & 3;
                *reinterpret_cast<float4*>(zstage + v * 16 + 4 * q) =
                    *reinterpret_cast<const float4*>(G + (size_t)v * gld + i0 + 4 * q);
            }
            __syncwarp();
        }
        for (int c0 = 0; c0 < jend; c0 += 64) {
            const int ngroups = min(4, (jend - c0 + 15) >> 4);
            prefetch_next();
            // ---- the tile's increment: sum over the pending vectors of z[row] * z[column] -------------------------
            float acc[8][4];
#pragma unroll
            for (int n = 0; n < 8; ++n) { acc[n][0] = 0.f; acc[n][1] = 0.f; acc[n][2] = 0.f; acc[n][3] = 0.f; }
            // one step: 8 pending vectors (this lane: vectors k0 = 8 ks + t and k0 + 4) times the tile's rows and columns
            auto kstep = [&](const float (&av)[4], const float2 (&b0)[4], const float2 (&b1)[4]) {
                uint32_t ah[4], al[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) tf32_split(av[q], ah[q], al[q]);
                uint32_t bh[8][2], bl[8][2];                              // the 8 MMA tiles: (k0, k1) parts
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    tf32_split2(b0[u], bh[2 * u][0], bh[2 * u + 1][0], bl[2 * u][0], bl[2 * u + 1][0]);
                    tf32_split2(b1[u], bh[2 * u][1], bh[2 * u + 1][1], bl[2 * u][1], bl[2 * u + 1][1]);
                }
                // The tensor core rounds every result toward zero (measured: the products of one instruction are
                // summed with guard bits, then truncated to FP32).  On a running accumulator that is a bias of about
                // 2^-25 of the accumulator per instruction, of the same sign for all d_col / 8 instructions of an
                // element.  So the three products of 8 pending vectors are summed from zero, the two small ones
                // first -- one truncation at the size of that partial sum -- and the partial sums are added to the
                // running increment in FP32 with round-to-nearest.  A product into an accumulator is issued eight
                // products after the previous one into it: their latency is long.
                float dk[8][4];
#pragma unroll
                for (int n = 0; n < 8; ++n) mma_tf32_z(dk[n], al, bh[n][0], bh[n][1]);
#pragma unroll
                for (int n = 0; n < 8; ++n) mma_tf32(dk[n], ah, bl[n][0], bl[n][1]);
#pragma unroll
                for (int n = 0; n < 8; ++n) mma_tf32(dk[n], ah, bh[n][0], bh[n][1]);
                // That one truncation per partial sum still shortens every increment by half a unit in the last place on
                // average, the same way for every element and pass -- a uniform scaling of all Lemma-1 updates, which the
                // last steps of a row (the few remaining entries carry everything eliminated before) amplify: measured
                // on a 2304-column layer, the final loss was off by 1.7e-4 with it and 1.3e-5 without.  Setting the last
                // mantissa bit turns "truncated" into "truncated + 0 or 1 unit", which is right on average.
#pragma unroll
                for (int n = 0; n < 8; ++n)
#pragma unroll
                    for (int e = 0; e < 4; e += 2) {                     // (two additions per instruction)
                        const float2 r = __fadd2_rn(make_float2(acc[n][e], acc[n][e + 1]),
                                                    make_float2(__uint_as_float(__float_as_uint(dk[n][e]) | 1u),
                                                                __uint_as_float(__float_as_uint(dk[n][e + 1]) | 1u)));
                        acc[n][e] = r.x; acc[n][e + 1] = r.y;
                    }
            };
            // column operands of an overflow step, straight from L2; issued one step ahead of their use
            float2 pb0[4], pb1[4];
            auto load_g = [&](int kg) {
                const int k0 = (kg << 3) + t, k1 = k0 + 4;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c = c0 + (u << 4) + (g << 1);               // < round_up(m1, 16) <= gld
                    pb0[u] = make_float2(0.f, 0.f); pb1[u] = pb0[u];
                    if (u < ngroups && k0 < nbg) pb0[u] = *reinterpret_cast<const float2*>(G + (size_t)k0 * gld + c);
                    if (u < ngroups && k1 < nbg) pb1[u] = *reinterpret_cast<const float2*>(G + (size_t)k1 * gld + c);
                }
            };
            if (GP && ksteps_g > 0) load_g(0);                            // in flight during the shared-memory steps
            for (int ks = 0; ks < ksteps; ++ks) {
                const int k0 = (ks << 3) + t, k1 = k0 + 4;
                const bool v0 = k0 < (GP ? nbs : nb), v1 = k1 < (GP ? nbs : nb);
                const float* z0 = Z + (size_t)k0 * ldz;
                const float* z1 = Z + (size_t)k1 * ldz;
                const float av[4] = {v0 && in[0] ? z0[rr[0]] : 0.f, v0 && in[1] ? z0[rr[1]] : 0.f,
                                     v1 && in[0] ? z1[rr[0]] : 0.f, v1 && in[1] ? z1[rr[1]] : 0.f};
                float2 b0[4], b1[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int c = c0 + (u << 4) + (g << 1);               // < m1 + 16 <= ldz
                    b0[u] = make_float2(0.f, 0.f); b1[u] = b0[u];         // (a group past the end multiplies zeros)
                    if (u < ngroups && v0) b0[u] = *reinterpret_cast<const float2*>(z0 + c);
                    if (u < ngroups && v1) b1[u] = *reinterpret_cast<const float2*>(z1 + c);
                }
                kstep(av, b0, b1);
            }
            if (GP) for (int kg = 0; kg < ksteps_g; ++kg) {
                const int k0 = (kg << 3) + t, k1 = k0 + 4;
                const bool v0 = k0 < nbg, v1 = k1 < nbg;
                const float av[4] = {v0 ? zstage[k0 * 16 + g] : 0.f, v0 ? zstage[k0 * 16 + g + 8] : 0.f,      // (rows past m1
                                     v1 ? zstage[k1 * 16 + g] : 0.f, v1 ? zstage[k1 * 16 + g + 8] : 0.f};     // are never stored)
                float2 b0[4], b1[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) { b0[u] = pb0[u]; b1[u] = pb1[u]; }
                if (kg + 1 < ksteps_g) load_g(kg + 1);
                kstep(av, b0, b1);
            }
            // ---- the tile of H (in L2 by now: the cursor passed it two tiles ago), minus the increment -----------
            float4 hv[4][2];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    hv[u][h] = make_float4(0.f, 0.f, 0.f, 0.f);
                    const int j = c0 + (u << 4) + (t << 2);
                    if (u < ngroups && in[h] && j <= rr[h]) {
                        const float4* src = reinterpret_cast<const float4*>(Hp + (size_t)sr[h] * ldp + j);
                        hv[u][h] = STREAM ? __ldcs(src) : *src;
                    }
                }
            // columns of this lane that are holes: their data sits in the mover's row
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (u < ngroups) {
                    const int j = c0 + (u << 4) + (t << 2);
                    const uint32_t my4 = (colmask[j >> 5] >> (j & 31)) & 0xFu;
                    if (my4) {
#pragma unroll
                        for (int comp = 0; comp < 4; ++comp) {
                            if (!((my4 >> comp) & 1u)) continue;
                            const int jj = j + comp;
                            const int sj = (int)srcm[jj];
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                if (in[h] && jj <= rr[h]) {
                                    const float val = Hp[(size_t)max(sr[h], sj) * ldp + min(sr[h], sj)];
                                    if (comp == 0) hv[u][h].x = val; else if (comp == 1) hv[u][h].y = val;
                                    else if (comp == 2) hv[u][h].z = val; else hv[u][h].w = val;
                                }
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (u < ngroups) {
                    const int j = c0 + (u << 4) + (t << 2);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (in[h] && j <= rr[h]) {
                            float4 o = hv[u][h];
                            o.x -= acc[2 * u][2 * h];     o.z -= acc[2 * u][2 * h + 1];
                            o.y -= acc[2 * u + 1][2 * h]; o.w -= acc[2 * u + 1][2 * h + 1];
                            float4* dst = reinterpret_cast<float4*>(Hp + (size_t)rr[h] * ldp + j);
                            if (STREAM) __stcs(dst, o); else *dst = o;
                        }
                    }
                }
            }
        }
    }
}

// Step-by-step Lemma-1 update on the shared-memory triangle S (leading dimension lds) in the coordinates
// that hold after slot `last` moved into slot pm (pm < 0: nothing moved); mp = rows left.
template <int NT>
__device__ __forceinline__ void blk_pass_shared(float* S, int lds, int mp, int pm, const float* v, const float* u,
                                                const float* lr) {
    constexpr int NW = NT / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = warp; i < mp; i += NW) {
        float* row = S + i * lds;
        const float nv = -v[i];
        for (int j = lane; j <= i; j += 32) {
            const float base = (i == pm) ? lr[j] : (j == pm ? lr[i] : row[j]);
            row[j] = fmaf(nv, u[j], base);
        }
    }
}

// Block pruning (Section 3, "Block-Sparsity", Eq. 5), blocks of 4: score w_P^T ((Hinv)_P)^-1 w_P of one 4-slot group
// from its weights w, the diagonal a_ii and the off-diagonals o = (a01, a02, a03, a12, a13, a23) of its 4 x 4 block, by
// an LDL^T factorisation: the score is sum_i y_i^2 / d_i, which is also the sum of the four single-weight losses
// when the members are eliminated in this order.  Returns NaN if the block is not positive definite.
__device__ __forceinline__ double block4_score(const double* w, const double* a, const double* o) {
    const double d0 = a[0], r0 = 1.0 / d0;
    const double l10 = o[0] * r0, l20 = o[1] * r0, l30 = o[2] * r0;
    const double d1 = a[1] - l10 * o[0], r1 = 1.0 / d1;
    const double t21 = o[3] - l20 * o[0], t31 = o[4] - l30 * o[0];
    const double l21 = t21 * r1, l31 = t31 * r1;
    const double d2 = a[2] - l20 * o[1] - l21 * t21, r2 = 1.0 / d2;
    const double t32 = o[5] - l30 * o[1] - l31 * t21;
    const double l32 = t32 * r2;
    const double d3 = a[3] - l30 * o[2] - l31 * t31 - l32 * t32, r3 = 1.0 / d3;
    const double y0 = w[0];
    const double y1 = w[1] - l10 * y0;
    const double y2 = w[2] - l20 * y0 - l21 * y1;
    const double y3 = w[3] - l30 * y0 - l31 * y1 - l32 * y2;
    if (!(d0 > 0.0) || !(d1 > 0.0) || !(d2 > 0.0) || !(d3 > 0.0)) return CUDART_NAN;
    return y0 * y0 * r0 + y1 * y1 * r1 + y2 * y2 * r2 + y3 * y3 * r3;
}

// Blocks of 8: the same score by Gaussian elimination of the members in ascending order on a copy of the 8 x 8 block
// (diagonal a, off-diagonals o packed by rows of the upper triangle: (0,1) .. (0,7), (1,2) .. (6,7)): the sum of the
// eight single-weight losses w_i^2 / a_ii met on the way.  Returns NaN if a pivot is not positive.
__device__ __forceinline__ int block8_index(int i, int j) { return i * (15 - i) / 2 + (j - i - 1); }      // i < j
__device__ __noinline__ double block8_score(const double* w, const double* a, const double* o) {
    double m[8][8], y[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        y[i] = w[i]; m[i][i] = a[i];
#pragma unroll
        for (int j = i + 1; j < 8; ++j) m[i][j] = o[block8_index(i, j)];
    }
    double sc = 0.0;
    bool ok = true;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const double dii = m[i][i], r = 1.0 / dii;
        ok = ok && (dii > 0.0);
        sc += y[i] * y[i] * r;
#pragma unroll
        for (int j = i + 1; j < 8; ++j) {
            const double l = m[i][j] * r;
            y[j] -= l * y[i];
#pragma unroll
            for (int k = j; k < 8; ++k) m[j][k] -= l * m[i][k];
        }
    }
    return ok ? sc : CUDART_NAN;
}

// Q = the kernel contains the OBQ code (modes QUANT and REPLAY_QUANT); the pruning kernels are built without it.
// BC = 4 or 8: block pruning in blocks of that many consecutive columns (pruning kernels only), 0: single weights.
// FG = the kernel takes forced eliminations (replay of a known order) four at a time: their order is known, so the
// four pivot columns are fetched and corrected together, the 4 x 4 block of the columns at the pivot slots is
// broadcast, and every thread carries out the four Lemma-1 eliminations on its own slots in registers -- two
// barriers per four steps, each pending vector read once for four columns.  Same arithmetic per element as four
// single steps except that a column's corrections are subtracted one by one instead of summed first.
// GPV = the kernel can keep further pending vectors in global memory (very long rows, 512 threads only).
// SH = the kernel takes shares of rows (a row may be started by one block and finished by the next); launches whose
// rows divide evenly over the blocks run the kernel built without that code.
template <int NT, int KMAX, bool Q, int BC, bool FG, bool GPV, bool SH>
__global__ void __launch_bounds__(NT, 512 / NT) blocked_engine_kernel(const EngineArgs a) {
    extern __shared__ __align__(16) char smem[];
    constexpr int NW = NT / 32;
    constexpr int BCD = BC ? BC : 1;                           // divisor that is never zero
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d = a.d, cap = a.cap, ms = a.ms;
    char* scratch = smem;
    Bcast* bc = reinterpret_cast<Bcast*>(smem + BLK_OFF_BC);
    int* pv = reinterpret_cast<int*>(smem + BLK_OFF_PV);
    int* hl = reinterpret_cast<int*>(smem + BLK_OFF_HL);
    int* mv = reinterpret_cast<int*>(smem + BLK_OFF_MV);
    float* rf = reinterpret_cast<float*>(smem + BLK_OFF_RF);
    uint32_t* colmask = reinterpret_cast<uint32_t*>(smem + BLK_OFF_CM);
    double* wd = reinterpret_cast<double*>(smem + BLK_FIXED);
    double* dg = wd + cap;
    int* perm = reinterpret_cast<int*>(dg + cap);
    unsigned short* srcm = reinterpret_cast<unsigned short*>(perm + cap);
    const bool has_wfull = a.w_trace != nullptr;
    float* wfull = reinterpret_cast<float*>(smem + BLK_FIXED + blk_state_bytes(cap, false));
    const bool has_nm = a.nm_prune > 0;                         // N:M pattern: at most nm_prune eliminations per block
    const int nm_lg = a.nm_lg, nm_prune = a.nm_prune;
    unsigned char* blkcnt = reinterpret_cast<unsigned char*>(smem + BLK_FIXED + blk_state_bytes(cap, has_wfull));
    double* boff = reinterpret_cast<double*>(smem + BLK_FIXED + blk_state_bytes(cap, has_wfull, has_nm));
    float* panel = reinterpret_cast<float*>(smem + BLK_FIXED + blk_state_bytes(cap, has_wfull, has_nm, BC));
    // tail views (step-by-step phase in shared memory) share the panel's space
    const int msr = (ms + 3) & ~3;
    float* tv = panel;
    float* tu = tv + msr;
    float* tlr = tu + msr;
    float* S = tlr + msr;
    const int lds = ms + 1;
    const int ldp = a.ldp;
    float* const Hp0 = a.Hws ? a.Hws + (size_t)blockIdx.x * d * a.ldp : nullptr;      // the block's own triangle
#define HP (SH ? (a.Hws + (size_t)reinterpret_cast<const int*>(smem + BLK_OFF_SCHED)[2] * d * ldp) : Hp0)
    // overflow of the pending vectors: gB more of them in global memory (sized to stay in L2), stride gld
    // (only the one-row-per-SM configuration uses it; the other kernels are built without that code)
    constexpr bool GP = GPV;
    const int gB = (GP && a.Gpan) ? a.g_vectors : 0, gld = a.g_ld;
    // (recomputed at every use instead of held in registers: the kernels with the overflow code have none to spare)
#define GVEC (a.Gpan + (size_t)blockIdx.x * a.g_vectors * a.g_ld)
#define ZSTAGE (panel + a.panel_floats + (size_t)warp * a.g_vectors * 16)      /* per warp: g_vectors x 16 floats */

    // ---- this block's items: whole rows, plus (shares of rows) the start of one row and the rest of another -------
    int* sched = reinterpret_cast<int*>(smem + BLK_OFF_SCHED);
    if (SH) {                                  // the item counter lives in shared memory too
        if (tid == 0) sched[3] = 0;
        __syncthreads();
    }
    for (int it_reg = 0;; ++it_reg) {
        int rr, kind, head_num;
        const int it = SH ? sched[3] : it_reg;
        if (SH) { __syncthreads(); if (tid == 0) sched[3] = it + 1; __syncthreads(); }    // read by all, then moved on
        if (!blk_item(SH, blockIdx.x, gridDim.x, a.row_count, it, &rr, &kind, &head_num)) break;
        const int NG = gridDim.x;
        const int r = a.row_begin + rr;
        // the triangle of the row in work: buffer blk for whole rows, ng + blk for the row this block starts, ng + blk - 1
        // for the row it finishes (kept in shared memory and re-read where needed, not in registers)
        int hbuf = kind == ITEM_FULL ? (int)blockIdx.x : (kind == ITEM_HEAD ? NG + (int)blockIdx.x : NG + (int)blockIdx.x - 1);
        int n_forced = 0, n_free = 0;
        bool quant = false;
        if (a.mode == MODE_PRUNE) { n_free = a.steps; }
        else if (a.mode == MODE_REPLAY) { n_forced = a.forced_counts[r]; }
        else if (a.mode == MODE_QUANT) { n_free = d; quant = Q; }
        else { n_forced = a.forced_counts[r]; n_free = d - n_forced; quant = Q; }
        if (n_forced < 0) n_forced = 0;
        if (n_forced > d) n_forced = d;
        if (n_free > d - n_forced) n_free = d - n_forced;
        const int total = n_forced + n_free;
        const bool outliers = Q && quant && (a.flags & OBC_FLAG_OUTLIERS);

        // ---- shares of rows: where this item stops, and what a continued row starts from -----------------
        int s_stop = total;                // steps [s_begin, s_stop) of the row are this item's
        int s_begin = 0, m_begin = d;
        if (kind == ITEM_HEAD) s_stop = blk_cut_step(d, ms, total, a.panel_floats, a.max_pending, gB, head_num, NG, blk_step_cost(NT));
        if (kind == ITEM_HEAD && s_stop <= 0) {
            // too small a share to be worth a start: the neighbour takes the whole row
            if (tid == 0) blk_publish(a.split_state + (size_t)blockIdx.x * a.split_stride, a.split_flags + blockIdx.x, 0, d, 0);
            continue;
        }
        if (kind == ITEM_TAIL) {
            const SplitHeader* sh = reinterpret_cast<const SplitHeader*>(a.split_state + (size_t)(blockIdx.x - 1) * a.split_stride);
            if (tid == 0) bc->nh = blk_wait_flag(a.split_flags + blockIdx.x - 1);
            __syncthreads();
            const int ok = bc->nh;
            __syncthreads();
            if (!ok) {                     // the start of this row never arrived: report it, touch nothing else
                if (tid == 0) a.row_status[r] = -(int)OBC_ERR_TIMEOUT;
                continue;
            }
            if (sh->done) continue;        // finished (or failed and reported) by the block that started it
            s_begin = sh->s_cut; m_begin = sh->m0;
            if (s_begin == 0) { kind = ITEM_FULL; hbuf = (int)blockIdx.x; }    // never started: a whole row
        }

        if (SH) {                              // read during and after the row
            if (tid == 0) { sched[0] = kind; sched[1] = s_stop; sched[2] = hbuf; }
            __syncthreads();
        }

        // ---- row set-up ------------------------------------------------------------------------------
        if (kind == ITEM_TAIL) {
            // continue a row: state as saved at the flush boundary s_begin (slots [0, m_begin) all live, nothing pending)
            blk_state_copy(false, a.split_state + (size_t)(blockIdx.x - 1) * a.split_stride, cap, d, m_begin, NT, wd, dg, perm, srcm,
                           has_wfull ? wfull : nullptr);
            for (int k = tid; k < 160; k += NT) colmask[k] = 0u;
            if (tid == 0) {
                bc->sc = 1.0; bc->ze = 0.0; bc->mq = 0.0;
                if (a.mode == MODE_QUANT || (a.mode == MODE_REPLAY_QUANT && s_begin > n_forced)) {
                    bc->sc = (double)a.scale[r]; bc->ze = (double)a.zero[r];
                    bc->mq = (double)grid_maxq(a.bits, a.symmetric);
                }
            }
        } else {
        for (int j = tid; j < d; j += NT) {
            const float w = a.W[(size_t)r * a.ldw + j];
            wd[j] = (double)w;
            dg[j] = (double)a.Hinv[(size_t)j * a.ldhi + j];
            perm[j] = j;
            srcm[j] = (unsigned short)j;
            if (has_wfull) wfull[j] = w;
            if (a.codes) a.codes[(size_t)r * d + j] = -1;
            if (a.mask) a.mask[(size_t)r * d + j] = 1;
        }
        if (has_nm) for (int b = tid; b < (d >> nm_lg); b += NT) blkcnt[b] = 0;
        if (BC == 8) {
            for (int e = tid; e < (d >> 3) * 28; e += NT) {
                const int g = e / 28, k = e - g * 28;
                int ia = 0, rest = k;
                while (rest >= 7 - ia) { rest -= 7 - ia; ++ia; }
                const int ib = ia + 1 + rest;
                boff[e] = (double)a.Hinv[(size_t)(8 * g + ia) * a.ldhi + 8 * g + ib];
            }
        } else if (BC) {
            for (int e = tid; e < (d >> 2) * 6; e += NT) {
                const int g = e / 6, k = e - g * 6;
                const int ia = k < 3 ? 0 : (k < 5 ? 1 : 2), ib = k < 3 ? k + 1 : (k < 5 ? k - 1 : 3);
                boff[e] = (double)a.Hinv[(size_t)(4 * g + ia) * a.ldhi + 4 * g + ib];
            }
        }
        for (int k = tid; k < 160; k += NT) colmask[k] = 0u;
        for (int j = d + tid; j < cap; j += NT) perm[j] = -1;
        if (tid == 0) {
            bc->sc = 1.0; bc->ze = 0.0; bc->mq = 0.0;
            if (a.mode == MODE_QUANT) {
                bc->sc = (double)a.scale[r]; bc->ze = (double)a.zero[r];
                bc->mq = (double)grid_maxq(a.bits, a.symmetric);
            }
            a.row_status[r] = 0;
        }
        if (a.w_trace)
            for (int j = tid; j < d; j += NT)
                a.w_trace[((size_t)r * (a.trace_steps + 1)) * d + j] = a.W[(size_t)r * a.ldw + j];
        }
        bool tail = false;
        if (kind != ITEM_TAIL && d > ms && total > 0) {
            for (int i = warp; i < d; i += NW) {
                const float4* s4 = reinterpret_cast<const float4*>(a.Hinv + (size_t)i * a.ldhi);
                float4* d4 = reinterpret_cast<float4*>(HP + (size_t)i * ldp);
                const int n4 = (i >> 2) + 1;
                if (GP || (FG && NT >= 512)) {      // (kernels with no registers to spare: one load in flight)
                    for (int j4 = lane; j4 < n4; j4 += 32) d4[j4] = s4[j4];
                } else {
                    for (int j0 = lane; j0 < n4; j0 += 128) {      // four loads in flight per lane
                        float4 t[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) if (j0 + 32 * k < n4) t[k] = __ldg(s4 + j0 + 32 * k);
#pragma unroll
                        for (int k = 0; k < 4; ++k) if (j0 + 32 * k < n4) d4[j0 + 32 * k] = t[k];
                    }
                }
            }
        }
        __syncthreads();
        double gsc = bc->sc, gze = bc->ze, gmq = bc->mq;       // grid parameters of the row (registers)

        int m0 = m_begin;                // slots in use (tail phase: number of live slots)
        int nb = 0;                      // pending vectors
        int ldz = blk_ldz(m0);
        int scap = a.panel_floats / ldz;     // pending vectors that fit into shared memory at this row length
        int bcur = min(a.max_pending, scap + gB);
        if (BC) bcur &= ~(BC - 1);           // whole blocks between two flushes, so that 4-slot groups stay together
        int s = s_begin;
        bool failed = false;
        int blk_base = 0;                // block pruning: first slot and score of the block being eliminated
        double blk_score = 0.0;
        float sa[KMAX];                  // score estimates of the own slots, kept up to date by the update phase
        unsigned cntw[KMAX / 4];         // N:M: eliminations so far in the block of each own slot (one byte per slot)
#pragma unroll
        for (int g = 0; g < KMAX / 4; ++g) cntw[g] = 0u;
        bool sa_valid = false;
        double gisc = 1.0 / gsc;
        for (; s < total; ++s) {
            if (!tail) {
                if (d > ms && nb > 0 && (nb == bcur || m0 - nb <= ms || (SH && s == sched[1]))) {
                    // ---- flush: apply the pending vectors and compact to m1 slots ------------------------
                    __syncthreads();                           // the last step's vector and perm updates
                    const int m1 = m0 - nb;
                    if (tid == 0) {
                        int nh = 0, sp = m1;
                        for (int b = 0; b < nb; ++b) {
                            const int h = pv[b];
                            if (h < m1) {
                                while (sp < m0 - 1 && perm[sp] < 0) ++sp;
                                hl[nh] = h; mv[nh] = sp; ++sp; ++nh;
                            }
                        }
                        bc->nh = nh;
                    }
                    __syncthreads();
                    const int nh = bc->nh;
                    for (int idx = tid; idx < nh * nb; idx += NT) {
                        const int q = idx / nb, b = idx - q * nb;
                        float* zr = (!GP || b < scap) ? panel + (size_t)b * ldz : GVEC + (size_t)(b - scap) * gld;
                        zr[hl[q]] = zr[mv[q]];
                    }
                    if (tid < nh) {
                        const int h = hl[tid];
                        srcm[h] = (unsigned short)mv[tid];
                        atomicOr(&colmask[h >> 5], 1u << (h & 31));
                    }
                    __syncthreads();
                    if (!GP)
                        blk_flush_mma<NT, true, false>(HP, ldp, m1, nb, nb, panel, ldz, nullptr, 0, nullptr, srcm, colmask);      // evict-first at every row length (~1 %)
                    else
                        blk_flush_mma<NT, true, true>(HP, ldp, m1, nb, min(nb, scap), panel, ldz, GVEC, gld, ZSTAGE, srcm, colmask);
                    __syncthreads();
                    if (tid < nh) {
                        const int h = hl[tid], sv = mv[tid];
                        wd[h] = wd[sv]; dg[h] = dg[sv]; perm[h] = perm[sv];
                        if (BC == 4 && (h & 3) == 0)      // holes and movers are whole aligned groups in block mode
                            for (int k = 0; k < 6; ++k) boff[(h >> 2) * 6 + k] = boff[(sv >> 2) * 6 + k];
                        if (BC == 8 && (h & 7) == 0)
                            for (int k = 0; k < 28; ++k) boff[(h >> 3) * 28 + k] = boff[(sv >> 3) * 28 + k];
                        srcm[h] = (unsigned short)h;
                        colmask[h >> 5] = 0u;
                    }
                    m0 = m1; nb = 0;
                    sa_valid = false;
#pragma unroll
                    for (int k = 0; k < KMAX; ++k) sa[k] = CUDART_NAN_F;      // slots changed hands: not carried over
#pragma unroll
                    for (int g = 0; g < KMAX / 4; ++g) cntw[g] = 0u;
                    ldz = blk_ldz(m0);
                    scap = a.panel_floats / ldz;
                    bcur = min(a.max_pending, scap + gB);
                    if (BC) bcur &= ~(BC - 1);
                    __syncthreads();
                }
                if (SH && s == sched[1]) break;      // (shares of rows) the row is handed over here, everything applied
                if (m0 <= ms) {
                    // ---- move on chip: slots [0, m0) are all live here and the stored triangle is current
                    const float* src = (d > ms) ? HP : a.Hinv;
                    const int sld = (d > ms) ? ldp : a.ldhi;
                    for (int i = warp; i < m0; i += NW)
                        for (int j = lane; j <= i; j += 32) S[i * lds + j] = src[(size_t)i * sld + j];
                    tail = true;
                    __syncthreads();
                }
            }
            const bool forced = s < n_forced;
            const bool q_now = Q && quant && !forced;
            if (FG && forced && !tail && !has_wfull && !has_nm && s + BLK_GS <= (SH ? min(n_forced, sched[1]) : n_forced) && nb + BLK_GS <= bcur &&
                (!GP || nb + BLK_GS <= scap)) {
                // ======================= four forced eliminations together ================================
                constexpr int GS = BLK_GS;
                int* gslot = reinterpret_cast<int*>(smem + BLK_OFF_GRP);
                float* gM = reinterpret_cast<float*>(smem + BLK_OFF_GRP + 16);
                int fo[GS];
#pragma unroll
                for (int g = 0; g < GS; ++g) fo[g] = a.forced_order[(size_t)r * d + s + g];
                unsigned live = 0u;
#pragma unroll
                for (int g4 = 0; g4 < KMAX / 4; ++g4) {
                    const int jb = own_slot<NT>(4 * g4);
                    if (jb >= m0) continue;
                    const int4 pm = *reinterpret_cast<const int4*>(perm + jb);
                    const int pq[4] = {pm.x, pm.y, pm.z, pm.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (jb + q < m0 && pq[q] >= 0) {
                            live |= 1u << (4 * g4 + q);
#pragma unroll
                            for (int g = 0; g < GS; ++g)
                                if (pq[q] == fo[g]) gslot[g] = jb + q;
                        }
                }
                __syncthreads();
                int p4[GS];
                bool ok = true;
#pragma unroll
                for (int g = 0; g < GS; ++g) {
                    p4[g] = gslot[g];
                    ok = ok && p4[g] >= 0 && p4[g] < m0 && perm[p4[g]] == fo[g];     // a stale entry never matches
                }
                ok = ok && p4[0] != p4[1] && p4[0] != p4[2] && p4[0] != p4[3] && p4[1] != p4[2] && p4[1] != p4[3] &&
                     p4[2] != p4[3];
                if (ok) {
                    double wp4[GS], dp4[GS];
#pragma unroll
                    for (int g = 0; g < GS; ++g) { wp4[g] = wd[p4[g]]; dp4[g] = dg[p4[g]]; }
                    // the four pivot columns of the stored matrix at the own slots
                    float v[GS][KMAX];
#pragma unroll
                    for (int g4 = 0; g4 < KMAX / 4; ++g4) {
                        const int jb = own_slot<NT>(4 * g4);
#pragma unroll
                        for (int g = 0; g < GS; ++g)
#pragma unroll
                            for (int q = 0; q < 4; ++q) v[g][4 * g4 + q] = 0.f;
                        if (jb >= m0) continue;
#pragma unroll
                        for (int g = 0; g < GS; ++g) {
                            const int p = p4[g];
                            const float* rowp = HP + (size_t)p * ldp;
                            if (jb + 3 <= p) {
                                const float4 t = *reinterpret_cast<const float4*>(rowp + jb);
                                v[g][4 * g4] = t.x; v[g][4 * g4 + 1] = t.y; v[g][4 * g4 + 2] = t.z; v[g][4 * g4 + 3] = t.w;
                            } else {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    const int j = jb + q;
                                    if ((live >> (4 * g4 + q)) & 1u) v[g][4 * g4 + q] = (j <= p) ? rowp[j] : HP[(size_t)j * ldp + p];
                                }
                            }
                        }
                    }
                    // corrected by the pending vectors (all of them in shared memory here)
                    for (int b = 0; b < nb; ++b) {
                        const float* zo = panel + (size_t)b * ldz;
                        float zp[GS];
#pragma unroll
                        for (int g = 0; g < GS; ++g) zp[g] = zo[p4[g]];
#pragma unroll
                        for (int g4 = 0; g4 < KMAX / 4; ++g4) {
                            if ((live >> (4 * g4)) & 0xFu) {
                                const float4 z = *reinterpret_cast<const float4*>(zo + own_slot<NT>(4 * g4));
#pragma unroll
                                for (int g = 0; g < GS; ++g) {
                                    v[g][4 * g4] = fmaf(-z.x, zp[g], v[g][4 * g4]);
                                    v[g][4 * g4 + 1] = fmaf(-z.y, zp[g], v[g][4 * g4 + 1]);
                                    v[g][4 * g4 + 2] = fmaf(-z.z, zp[g], v[g][4 * g4 + 2]);
                                    v[g][4 * g4 + 3] = fmaf(-z.w, zp[g], v[g][4 * g4 + 3]);
                                }
                            }
                        }
                    }
                    // the columns at the four pivot slots, from the owners of those slots
#pragma unroll
                    for (int k = 0; k < KMAX; ++k) {
                        if (!((live >> k) & 1u)) continue;
                        const int j = own_slot<NT>(k);
#pragma unroll
                        for (int g2 = 0; g2 < GS; ++g2)
                            if (j == p4[g2]) {
#pragma unroll
                                for (int g = 0; g < GS; ++g) gM[g * GS + g2] = v[g][k];
                            }
                    }
                    __syncthreads();
                    // the four eliminations at the pivot slots themselves (every thread, same values)
                    float zz[GS][GS];                      // vector e at pivot slot x
                    double idp[GS], fg[GS];
                    float rsq[GS];
                    bool fine = true;
#pragma unroll
                    for (int g = 0; g < GS; ++g) {
                        float mc[GS];
#pragma unroll
                        for (int x = 0; x < GS; ++x) {
                            mc[x] = gM[g * GS + x];
#pragma unroll
                            for (int e = 0; e < g; ++e) mc[x] = fmaf(-zz[e][x], zz[e][g], mc[x]);
                        }
                        const double dpp = dp4[g], w = wp4[g];
                        if (!(dpp > 0.0) || !isfinite(dpp) || !isfinite(w)) fine = false;
                        idp[g] = 1.0 / dpp;
                        fg[g] = w * idp[g];
                        rsq[g] = __frsqrt_rn((float)dpp);
#pragma unroll
                        for (int x = 0; x < GS; ++x) zz[g][x] = mc[x] * rsq[g];
#pragma unroll
                        for (int x = g + 1; x < GS; ++x) {
                            wp4[x] -= fg[g] * (double)mc[x];
                            dp4[x] -= (double)mc[x] * (double)mc[x] * idp[g];
                        }
                    }
                    if (fine) {
#pragma unroll
                        for (int g4 = 0; g4 < KMAX / 4; ++g4) {
                            const int jb = own_slot<NT>(4 * g4);
                            if (jb >= m0) continue;
                            float zv[GS][4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int k = 4 * g4 + q, j = jb + q;
#pragma unroll
                                for (int g = 0; g < GS; ++g) zv[g][q] = 0.f;
                                if (!((live >> k) & 1u)) continue;
                                int gm = GS;                   // this slot is the gm-th pivot (GS: none of them)
#pragma unroll
                                for (int g = 0; g < GS; ++g) if (j == p4[g]) gm = g;
                                double nw = wd[j], nd = dg[j];
#pragma unroll
                                for (int g = 0; g < GS; ++g) {
                                    if (g < gm) {
                                        float vj = v[g][k];
#pragma unroll
                                        for (int e = 0; e < g; ++e) vj = fmaf(-zv[e][q], zz[e][g], vj);
                                        nw -= fg[g] * (double)vj;
                                        nd -= (double)vj * (double)vj * idp[g];
                                        zv[g][q] = vj * rsq[g];
                                    }
                                }
                                if (gm < GS) perm[j] = -1;
                                else { wd[j] = nw; dg[j] = nd; }
                            }
#pragma unroll
                            for (int g = 0; g < GS; ++g)
                                *reinterpret_cast<float4*>(panel + (size_t)(nb + g) * ldz + jb) =
                                    make_float4(zv[g][0], zv[g][1], zv[g][2], zv[g][3]);
                        }
                        if (tid < GS) {
                            pv[nb + tid] = p4[tid];
                            if (a.W_out) a.W_out[(size_t)r * a.ldwo + fo[tid]] = 0.f;
                            if (a.mask) a.mask[(size_t)r * d + fo[tid]] = 0;
                        }
                        nb += GS;
                        s += GS - 1;
                        sa_valid = false;
#pragma unroll
                        for (int k = 0; k < KMAX; ++k) sa[k] = CUDART_NAN_F;
                        continue;
                    }
                }
                // an entry of the order that is not live, or a pivot that is not positive: the single steps below
                // meet it again and report it
            }
            // ---- grid of the compound path: built from the survivors when the replay is over -----------
            if (Q && a.mode == MODE_REPLAY_QUANT && s == n_forced) {
                float lo = 0.f, hi = 0.f;
#pragma unroll
                for (int k = 0; k < KMAX; ++k) {               // own slots: their owner is the only writer
                    const int j = own_slot<NT>(k);
                    if (j < m0 && perm[j] >= 0) { const float w = (float)wd[j]; lo = fminf(lo, w); hi = fmaxf(hi, w); }
                }
#pragma unroll
                for (int off = 16; off; off >>= 1) {
                    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, off));
                    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, off));
                }
                if (lane == 0) { rf[warp] = lo; rf[32 + warp] = hi; }
                __syncthreads();
                for (int k = 0; k < NW; ++k) { lo = fminf(lo, rf[k]); hi = fmaxf(hi, rf[32 + k]); }
                float sc, ze;
                grid_from_range(lo, hi, a.bits, a.symmetric, &sc, &ze);
                if (tid == 0) { a.scale[r] = sc; a.zero[r] = ze; }
                gsc = (double)sc; gze = (double)ze; gmq = (double)grid_maxq(a.bits, a.symmetric);
                gisc = 1.0 / gsc;
                sa_valid = false;
                __syncthreads();                               // rf is reused by the next row's grid
            }
            // ---- pick the slot: one candidate per thread, combined through the record buffer ------------
            unsigned key = KEY_NONE;
            double cs = 0.0;
            int cslot = -1;
            if (forced) {
                const int f = a.forced_order[(size_t)r * d + s];
#pragma unroll
                for (int k = 0; k < KMAX; ++k) {
                    const int j = own_slot<NT>(k);
                    if (j < m0 && perm[j] == f) { cslot = j; key = 0x80000000u; }
                }
            } else if (BC && (s - n_forced) % BCD != 0) {
                // the next member of the block chosen at the last block boundary
                const int j = blk_base + (s - n_forced) % BCD;
                if (j >= (tid << 2) && ((j - (tid << 2)) % (4 * NT)) < 4) { cslot = j; key = 0x80000000u; }
            } else if (BC) {
                // block boundary: exact FP64 score of every own live group (its four slots are all live here)
                double bs = CUDART_INF;
                int bo = 0x7fffffff;
#pragma unroll
                for (int g = 0; g < KMAX / 4; ++g) {
                    const int jb = own_slot<NT>(4 * g);
                    if (BC == 8 && (jb & 7) != 0) continue;      // a block of 8 is scored by the owner of its first half
                    if (jb < m0 && perm[jb] >= 0) {
                        const double sc4 = BC == 8 ? block8_score(wd + jb, dg + jb, boff + (jb >> 3) * 28)
                                                   : block4_score(wd + jb, dg + jb, boff + (jb >> 2) * 6);
                        const int o = perm[jb];
                        if (key_less(sc4, o, bs, bo)) { bs = sc4; bo = o; cslot = jb; }
                    }
                }
                cs = bs;
                if (cslot >= 0) key = float_key(__double2float_rn(bs));
            } else {
                if (!sa_valid || tail || outliers)
                    estimate_own<NT, KMAX, Q>(sa, wd, dg, perm, m0, q_now, gsc, gisc, gze, gmq, has_nm ? blkcnt : nullptr,
                                           nm_lg, nm_prune, cntw);
                thread_best<NT, KMAX, Q>(sa, wd, dg, perm, q_now, outliers, gsc, gisc, gze, gmq, &key, &cs, &cslot);
            }
            const Records rec = rec_view(scratch, s & 1);
            const Pick pk = block_pick<NT>(key, cs, cslot, cslot >= 0 ? perm[cslot] : -1,
                                           cslot >= 0 ? wd[cslot] : 0.0, cslot >= 0 ? dg[cslot] : 0.0, rec);
            const int p = pk.slot, op = pk.orig;
            const double dpp = pk.dgv, wp = pk.w;
            if (BC && !forced && (s - n_forced) % BCD == 0) { blk_base = p; blk_score = pk.s; }
            if (p < 0 || !(dpp > 0.0) || !isfinite(dpp) || !isfinite(wp)) { failed = true; break; }
            double qp = 0.0, code = -1.0;
            if (Q && q_now) qp = grid_q(wp, gsc, gze, gmq, &code);
            const double e = wp - qp;
            if (!tail) {
                // ======================= deferred-update step ==============================================
                float* zb = (!GP || nb < scap) ? panel + (size_t)nb * ldz : GVEC + (size_t)(nb - scap) * gld;
                // pivot column of the stored matrix (own slots), corrected by the pending vectors
                float c[KMAX], corr[KMAX];
                unsigned live = 0u;
                const float* rowp = HP + (size_t)p * ldp;
#pragma unroll
                for (int g = 0; g < KMAX / 4; ++g) {
                    const int jb = own_slot<NT>(4 * g);
#pragma unroll
                    for (int q = 0; q < 4; ++q) { c[4 * g + q] = 0.f; corr[4 * g + q] = 0.f; }
                    if (jb >= m0) continue;
                    const int4 pm = *reinterpret_cast<const int4*>(perm + jb);
                    const int pq[4] = {pm.x, pm.y, pm.z, pm.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (jb + q < m0 && pq[q] >= 0) live |= 1u << (4 * g + q);
                    if (jb + 3 <= p) {
                        const float4 v = *reinterpret_cast<const float4*>(rowp + jb);
                        c[4 * g] = v.x; c[4 * g + 1] = v.y; c[4 * g + 2] = v.z; c[4 * g + 3] = v.w;
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int j = jb + q;
                            if ((live >> (4 * g + q)) & 1u) c[4 * g + q] = (j <= p) ? rowp[j] : HP[(size_t)j * ldp + p];
                        }
                    }
                }
                const double idpp = 1.0 / dpp;
                const double f = e * idpp;
                const float rs = __frsqrt_rn((float)dpp);
                const int nbs = GP ? min(nb, scap) : nb;
                for (int b = 0; b < nbs; ++b) {
                    const float* zo = panel + (size_t)b * ldz;
                    const float zp = zo[p];
#pragma unroll
                    for (int g = 0; g < KMAX / 4; ++g) {
                        if ((live >> (4 * g)) & 0xFu) {
                            const float4 z = *reinterpret_cast<const float4*>(zo + own_slot<NT>(4 * g));
                            corr[4 * g] = fmaf(z.x, zp, corr[4 * g]);
                            corr[4 * g + 1] = fmaf(z.y, zp, corr[4 * g + 1]);
                            corr[4 * g + 2] = fmaf(z.z, zp, corr[4 * g + 2]);
                            corr[4 * g + 3] = fmaf(z.w, zp, corr[4 * g + 3]);
                        }
                    }
                }
                if (GP)
#pragma unroll 2
                for (int b = nbs; b < nb; ++b) {               // the overflow vectors, from L2
                    const float* zo = GVEC + (size_t)(b - scap) * gld;
                    const float zp = zo[p];
#pragma unroll
                    for (int g = 0; g < KMAX / 4; ++g) {
                        if ((live >> (4 * g)) & 0xFu) {
                            const float4 z = *reinterpret_cast<const float4*>(zo + own_slot<NT>(4 * g));
                            corr[4 * g] = fmaf(z.x, zp, corr[4 * g]);
                            corr[4 * g + 1] = fmaf(z.y, zp, corr[4 * g + 1]);
                            corr[4 * g + 2] = fmaf(z.z, zp, corr[4 * g + 2]);
                            corr[4 * g + 3] = fmaf(z.w, zp, corr[4 * g + 3]);
                        }
                    }
                }
                // state update of the own slots (Eq. 3 / Eq. 7), the new pending vector, and the score
                // estimates the next free step starts from
                const bool est_next = !BC && (s + 1 >= n_forced) && !outliers;
                const bool q_next = Q && quant && (s + 1 >= n_forced);
#pragma unroll
                for (int g = 0; g < KMAX / 4; ++g) {
                    const int jb = own_slot<NT>(4 * g);
                    if (jb >= m0) continue;
                    const int4 pm = *reinterpret_cast<const int4*>(perm + jb);
                    const int pq[4] = {pm.x, pm.y, pm.z, pm.w};
                    float zv[4];
                    // the group's FP64 state as 128-bit accesses: a warp's 64-bit accesses at this stride (32 bytes
                    // between lanes) would meet four to a bank; dead slots keep the value they had
                    double2* wq = reinterpret_cast<double2*>(wd + jb);
                    double2* dq = reinterpret_cast<double2*>(dg + jb);
                    const double2 w01 = wq[0], w23 = wq[1], d01 = dq[0], d23 = dq[1];
                    double wv[4] = {w01.x, w01.y, w23.x, w23.y}, dv[4] = {d01.x, d01.y, d23.x, d23.y};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int k = 4 * g + q, j = jb + q;
                        zv[q] = 0.f;
                        sa[k] = CUDART_NAN_F;
                        if (!((live >> k) & 1u)) continue;
                        if (j == p) {
                            perm[j] = -1;
                            if (has_nm) blkcnt[op >> nm_lg] += 1;      // read again only behind a barrier
                            continue;
                        }
                        const float vj = c[k] - corr[k];
                        const double nw = wv[q] - f * (double)vj;
                        const double nd = dv[q] - (double)vj * (double)vj * idpp;
                        wv[q] = nw; dv[q] = nd;
                        zv[q] = vj * rs;
                        if (est_next) sa[k] = score_estimate<Q>(nw, nd, q_next, gsc, gisc, gze, gmq);
                        if (has_nm) {
                            if ((pq[q] >> nm_lg) == (op >> nm_lg)) cntw[g] += 1u << (8 * q);
                            if ((int)((cntw[g] >> (8 * q)) & 0xFFu) >= nm_prune) sa[k] = CUDART_NAN_F;
                        }
                        if (has_wfull) wfull[pq[q]] = (float)nw;
                    }
                    wq[0] = make_double2(wv[0], wv[1]); wq[1] = make_double2(wv[2], wv[3]);
                    dq[0] = make_double2(dv[0], dv[1]); dq[1] = make_double2(dv[2], dv[3]);
                    *reinterpret_cast<float4*>(zb + jb) = make_float4(zv[0], zv[1], zv[2], zv[3]);
                    if (BC == 4 && ((live >> (4 * g)) & 0xFu) == 0xFu && jb != (p & ~3)) {
                        // Lemma 1 on the group's own 4 x 4 diagonal block (off-diagonal part; dg holds the diagonal)
                        double* o = boff + (jb >> 2) * 6;
                        const double v0 = (double)(c[4 * g] - corr[4 * g]), v1 = (double)(c[4 * g + 1] - corr[4 * g + 1]);
                        const double v2 = (double)(c[4 * g + 2] - corr[4 * g + 2]), v3 = (double)(c[4 * g + 3] - corr[4 * g + 3]);
                        o[0] -= v0 * v1 * idpp; o[1] -= v0 * v2 * idpp; o[2] -= v0 * v3 * idpp;
                        o[3] -= v1 * v2 * idpp; o[4] -= v1 * v3 * idpp; o[5] -= v2 * v3 * idpp;
                    }
                }
                if (BC == 8) {
                    // Lemma 1 on the 8 x 8 diagonal block of every other whole block: its two halves belong to
                    // neighbouring lanes, which exchange their four column entries; the lane of the first half takes
                    // the pairs whose smaller index is 0 or 1, the other lane the rest
#pragma unroll
                    for (int g = 0; g < KMAX / 4; ++g) {
                        const int jb = own_slot<NT>(4 * g);
                        float mine[4], other[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) mine[q] = c[4 * g + q] - corr[4 * g + q];
#pragma unroll
                        for (int q = 0; q < 4; ++q) other[q] = __shfl_xor_sync(0xffffffffu, mine[q], 1);
                        if (jb < m0 && ((live >> (4 * g)) & 0xFu) == 0xFu && (jb & ~7) != (p & ~7)) {
                            const bool first = (jb & 7) == 0;
                            double v[8];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                v[q] = (double)(first ? mine[q] : other[q]);
                                v[4 + q] = (double)(first ? other[q] : mine[q]);
                            }
                            double* o = boff + (jb >> 3) * 28;
#pragma unroll
                            for (int i = 0; i < 7; ++i)
#pragma unroll
                                for (int j = i + 1; j < 8; ++j)
                                    if ((i < 2) == first) o[block8_index(i, j)] -= v[i] * v[j] * idpp;
                        }
                    }
                }
                sa_valid = est_next;
                if (tid == 0) {
                    pv[nb] = p;
                    if (has_wfull) wfull[op] = (float)qp;
                    if (a.W_out) a.W_out[(size_t)r * a.ldwo + op] = (float)qp;
                    if (a.mask) a.mask[(size_t)r * d + op] = 0;
                    if (!forced) {
                        const int t = s - n_forced;
                        if (a.order) a.order[(size_t)r * d + t] = op;
                        if (a.loss) a.loss[(size_t)r * d + t] = BC ? ((t % BCD) ? 0.f : (float)blk_score) : (float)(e * e / dpp);
                    }
                    if (q_now && a.codes) a.codes[(size_t)r * d + op] = (int)code;
                }
                ++nb;
                if (a.w_trace && s < a.trace_steps) {
                    __syncthreads();
                    for (int j = tid; j < d; j += NT)
                        a.w_trace[((size_t)r * (a.trace_steps + 1) + s + 1) * d + j] = wfull[j];
                    // wfull is next written in the update phase of the following step, i.e. behind that step's
                    // barrier, which every thread reaches only after these reads
                }
            } else {
                // ======================= on-chip step (compaction at every step) ===========================
                const int m = m0, last = m0 - 1;
                for (int j = tid; j < m; j += NT) {
                    tv[j] = (j <= p) ? S[p * lds + j] : S[j * lds + p];
                    tlr[j] = S[last * lds + j];
                }
                __syncthreads();
                {
                    const double f = e / dpp;
                    for (int j = tid; j < m; j += NT) {
                        if (j == p) continue;
                        const float vj = tv[j];
                        const double nw = wd[j] - f * (double)vj;
                        const double nd = dg[j] - (double)vj * (double)vj / dpp;
                        const float uj = (float)((double)vj / dpp);
                        const int oj = perm[j];
                        if (has_wfull) wfull[oj] = (float)nw;
                        const int dst = (j == last) ? p : j;       // p != last here
                        wd[dst] = nw; dg[dst] = nd; tu[dst] = uj;
                        if (j == last) { perm[p] = oj; tv[p] = vj; tlr[p] = tlr[last]; }
                    }
                    if (tid == 0) {
                        if (has_nm) blkcnt[op >> nm_lg] += 1;
                        if (a.mask) a.mask[(size_t)r * d + op] = 0;
                        if (has_wfull) wfull[op] = (float)qp;
                        if (a.W_out) a.W_out[(size_t)r * a.ldwo + op] = (float)qp;
                        if (!forced) {
                            const int t = s - n_forced;
                            if (a.order) a.order[(size_t)r * d + t] = op;
                            if (a.loss) a.loss[(size_t)r * d + t] = (float)(e * e / dpp);
                        }
                        if (q_now && a.codes) a.codes[(size_t)r * d + op] = (int)code;
                    }
                }
                __syncthreads();
                if (a.w_trace && s < a.trace_steps)
                    for (int j = tid; j < d; j += NT)
                        a.w_trace[((size_t)r * (a.trace_steps + 1) + s + 1) * d + j] = wfull[j];
                const int pm = (p == last) ? -1 : p;
                if (s + 1 < total) blk_pass_shared<NT>(S, lds, m - 1, pm, tv, tu, tlr);
                --m0;
                __syncthreads();
            }
        }
        // ---- row epilogue ---------------------------------------------------------------------------------
        __syncthreads();
        if (SH && sched[0] == ITEM_HEAD) {
            // (shares of rows) leave the row to the next block: state at the flush boundary, then the flag
            const bool handed = !failed && s < total;
            if (handed)
                blk_state_copy(true, a.split_state + (size_t)blockIdx.x * a.split_stride, cap, d, m0, NT, wd, dg, perm, srcm,
                               has_wfull ? wfull : nullptr);
            else
                __threadfence();
            __syncthreads();
            if (tid == 0)
                blk_publish(a.split_state + (size_t)blockIdx.x * a.split_stride, a.split_flags + blockIdx.x, s, m0, handed ? 0 : 1);
            if (handed) { __syncthreads(); continue; }
        }
        if (failed) {           // stopped early: report the step, mark what was not produced
            if (tid == 0) a.row_status[r] = 1 + s;
            const int t0 = (s < n_forced) ? 0 : s - n_forced;
            for (int t = t0 + tid; t < n_free; t += NT) {
                if (a.order) a.order[(size_t)r * d + t] = -1;
                if (a.loss) a.loss[(size_t)r * d + t] = CUDART_INF_F;
            }
        }
        if (a.W_out)            // eliminated entries were written at their step; the live ones follow here
            for (int j = tid; j < m0; j += NT)
                if (perm[j] >= 0) a.W_out[(size_t)r * a.ldwo + perm[j]] = (float)wd[j];
        __syncthreads();
    }
}

#undef HP
#undef GVEC
#undef ZSTAGE
// ---- host side ---------------------------------------------------------------------------------------------
struct BlkPlan {
    int nt;            // threads per block
    int per_sm;        // blocks per SM the shared-memory split is made for
    size_t smem;       // dynamic shared memory per block
    int panel_floats;
    int ms;
    int g_vectors;     // overflow pending vectors per block in global memory (0 = none)
    int g_ld;          // their stride in floats
};

constexpr size_t BLK_L2_PANEL_BUDGET = (size_t)48 << 20;      // all blocks' overflow vectors together: well inside L2

static int blk_pick_ms(int d, size_t panel_bytes) {
    int ms = d < 1024 ? d : 1024;
    if (ms < 2) ms = 2;
    while (ms > 2 && blk_tail_bytes(ms) > panel_bytes) --ms;
    return ms;
}

// Threads per block and blocks per SM by row length: short rows are bound by the latency of a step, so
// several of them share an SM; long rows need the shared memory for pending vectors.
// row_count = rows of the launch (0 = many).
static bool blk_plan(int d, bool wfull, const DeviceInfo& di, BlkPlan* out, bool nm = false, int bc = 0,
                     int row_count = 0, int threads = 0) {
    const int cap = (d + 3) & ~3;
    int nt = threads;
    if (nt != 128 && nt != 256 && nt != 512) {
        // measured on full waves of rows: 128 threads win up to d_col ~ 700, 256 up to ~ 1400, 512 above
        nt = d <= 704 ? 128 : (d <= 1408 ? 256 : 512);
        // few rows (one per SM pair at most): nothing to share an SM with, the larger block is faster per row
        if (nt == 128 && row_count > 0 && row_count <= 2 * di.sm_count) nt = 256;
        // at most one row per SM: from d_col ~ 1000 the whole SM on one row wins (1024: 7 %, 1280: 20 %)
        if (nt == 256 && row_count > 0 && row_count <= di.sm_count && d > 960) nt = 512;
    }
    if (nt == 128 && cap > 1024) nt = 256;
    if (nt == 256 && cap > 2048) nt = 512;
    BlkPlan p;
    p.nt = nt;
    p.per_sm = 512 / nt;
    // 1 KB per resident block is reserved by the hardware; keep every block's share 128-byte aligned
    const size_t sm_total = (size_t)di.smem_optin + 1024;
    size_t share = (sm_total / p.per_sm - 1024) & ~(size_t)127;
    if (share > (size_t)di.smem_optin) share = (size_t)di.smem_optin;
    const size_t fixed = BLK_FIXED + blk_state_bytes(cap, wfull, nm, bc);
    const size_t min_panel = (size_t)4 * blk_ldz(cap);
    const size_t min_vectors = bc > 4 ? (size_t)bc : 4;         // (block pruning flushes whole blocks of bc updates)
    while (p.per_sm > 1 && share < fixed + min_vectors * min_panel) {     // too little room: fewer, larger blocks
        p.per_sm >>= 1;
        share = (sm_total / p.per_sm - 1024) & ~(size_t)127;
        if (share > (size_t)di.smem_optin) share = (size_t)di.smem_optin;
    }
    if (share < fixed + min_panel || share < fixed + blk_tail_bytes(2)) return false;
    p.smem = share;
    p.panel_floats = (int)((share - fixed) / 4);
    p.ms = blk_pick_ms(d, share - fixed);
    // Very long rows (d_col > ~2600): shared memory holds fewer than 16 pending vectors, so a pass over the triangle
    // applies few updates; further vectors go to a global buffer small enough to stay in L2 (the triangle itself is
    // streamed past it with evict-first hints).  Measured at d_col = 3072: 99 -> 73 ms per wave of rows.  At 2304 (19
    // vectors in shared memory) 16 more gain 2 % on one wave of rows and lose 2 % when rows are handed over between
    // blocks (rows out of step with each other compete for L2), so it is not used there.
    p.g_ld = (cap + 15) & ~15;
    p.g_vectors = 0;
    if (p.nt == 512) {
        const int in_smem = p.panel_floats / blk_ldz(cap);
        int g = (int)(BLK_L2_PANEL_BUDGET / ((size_t)di.sm_count * p.g_ld * 4));
        if (g > 32) g = 32;
        g &= ~7;                                                   // the flush multiplies 8 vectors at a time
        const size_t stage = (size_t)(p.nt / 32) * g * 16 * 4;     // per-warp staging of their row operands
        if (in_smem < 16 && g >= 8 && share - fixed >= stage + 4 * min_panel) {
            p.g_vectors = g;
            p.panel_floats = (int)((share - fixed - stage) / 4);
            p.ms = blk_pick_ms(d, share - fixed - stage);
        }
    }
    *out = p;
    return true;
}

// The largest grid any thread-count choice uses at this row length (threads per row are bounded below by the row
// length, see blk_plan).
static int blk_max_blocks(int d, const DeviceInfo& di) {
    const int cap = (d + 3) & ~3;
    return di.sm_count * (cap > 2048 ? 1 : (cap > 1024 ? 2 : 4));
}

size_t blocked_engine_workspace_bytes(int row_count, int d, const DeviceInfo& di) {
    // valid for every per-call choice: a row needs its private triangle whenever d exceeds the on-chip threshold,
    // and that threshold depends on the threads per row and on the per-row state the call keeps
    bool off_chip = false;
    const int nts[4] = {0, 128, 256, 512};
    for (int k = 0; k < 4; ++k)
        for (int nm = 0; nm < 2; ++nm) {
            BlkPlan p;
            if (!blk_plan(d, true, di, &p, nm != 0, false, row_count, nts[k])) continue;
            if (d > p.ms) off_chip = true;
        }
    if (!off_chip) return 256;
    const int cap = (d + 3) & ~3;
    int blocks = blk_max_blocks(d, di);
    // more rows than blocks: every block may also hold the row it starts for its neighbour (a second triangle),
    // plus the saved state and the flags of the hand-over
    const bool may_split = row_count == 0 || row_count > di.sm_count;
    if (row_count > 0 && row_count < blocks) blocks = row_count;
    const int gblocks = blocks < di.sm_count ? blocks : di.sm_count;     // overflow vectors: one block per SM only
    return round_up((size_t)blocks * (may_split ? 2 : 1) * d * cap * sizeof(float), 256) +
           round_up((size_t)gblocks * BLK_MAXB * ((cap + 15) & ~15) * sizeof(float), 256) +
           (may_split ? round_up((size_t)blocks * blk_split_stride(cap), 256) + round_up((size_t)blocks * sizeof(int), 256) : 0);
}

obc_status blocked_engine_plan(int d, int with_trace, int row_count, const EngineOpts& eo, int32_t* plan) {
    DeviceInfo di;
    obc_status st = device_info(&di);
    if (st != OBC_OK) return st;
    BlkPlan p;
    if (d > OBC_MAX_DCOL || !blk_plan(d, with_trace != 0, di, &p, false, false, row_count, eo.threads)) return OBC_ERR_UNSUPPORTED;
    const int mp = eo.max_pending;
    plan[0] = OBC_ENGINE_BLOCKED; plan[1] = p.nt; plan[2] = p.per_sm; plan[3] = p.ms; plan[4] = p.panel_floats;
    plan[5] = (mp >= 1 && mp <= BLK_MAXB) ? mp : BLK_MAXB; plan[6] = di.sm_count; plan[7] = p.g_vectors;
    return OBC_OK;
}

template <int NT, int KMAX, bool Q, int BC, bool FG, bool GPV>
static obc_status blk_launch_g(EngineArgs a, int blocks, size_t smem, int sm_count, cudaStream_t stream) {
    auto kernel = blocked_engine_kernel<NT, KMAX, Q, BC, FG, GPV, false>;
    auto kernel_sh = blocked_engine_kernel<NT, KMAX, Q, BC, FG, GPV, (BC == 0)>;     // (block pruning takes no shares)
    if (a.split) {
        // A block may wait (bounded) for the row its neighbour started, so all blocks must be resident at once: checked
        // here, and guaranteed by a cooperative launch.  If the grid does not fit, rows run in whole waves instead.
        OBC_CUDA_TRY(cudaFuncSetAttribute(kernel_sh, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        int per_sm = 0;
        OBC_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel_sh, NT, smem));
        int coop = 0, dev = 0;
        OBC_CUDA_TRY(cudaGetDevice(&dev));
        OBC_CUDA_TRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
        if (BC != 0 || !coop || (long long)per_sm * sm_count < blocks) a.split = 0;
    }
    if (a.split) {
        OBC_CUDA_TRY(cudaMemsetAsync(a.split_flags, 0, (size_t)blocks * sizeof(int), stream));
        void* params[1] = {(void*)&a};
        OBC_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)kernel_sh, dim3(blocks), dim3(NT), params, smem, stream));
    } else {
        OBC_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        kernel<<<blocks, NT, smem, stream>>>(a);
    }
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

template <int NT, int KMAX, bool Q, int BC, bool FG>
static obc_status blk_launch_q(const EngineArgs& a, int blocks, size_t smem, int sm_count, cudaStream_t stream) {
    if (NT >= 512 && a.Gpan != nullptr) return blk_launch_g<NT, KMAX, Q, BC, FG, (NT >= 512)>(a, blocks, smem, sm_count, stream);
    return blk_launch_g<NT, KMAX, Q, BC, FG, false>(a, blocks, smem, sm_count, stream);
}

template <int NT, int KMAX>
static obc_status blk_launch(const EngineArgs& a, int blocks, size_t smem, int sm_count, cudaStream_t stream) {
    if (a.block_c == 4) return blk_launch_q<NT, KMAX, false, 4, false>(a, blocks, smem, sm_count, stream);
    if (a.block_c == 8) return blk_launch_q<NT, KMAX, false, 8, false>(a, blocks, smem, sm_count, stream);
    switch (a.mode) {                       // the replay modes are the ones with forced eliminations
        case MODE_QUANT:        return blk_launch_q<NT, KMAX, true, 0, false>(a, blocks, smem, sm_count, stream);
        // (with 512 threads the OBQ kernel has no registers to spare for the four columns: single steps there)
        case MODE_REPLAY_QUANT: return blk_launch_q<NT, KMAX, true, 0, (NT <= 256)>(a, blocks, smem, sm_count, stream);
        case MODE_REPLAY:       return blk_launch_q<NT, KMAX, false, 0, true>(a, blocks, smem, sm_count, stream);
        default:                return blk_launch_q<NT, KMAX, false, 0, false>(a, blocks, smem, sm_count, stream);
    }
}
static obc_status blk_launch_nt(const EngineArgs& a, int nt, int blocks, size_t smem, int sm_count, cudaStream_t stream);

obc_status blocked_engine_launch(EngineArgs a, void* ws, size_t ws_bytes, cudaStream_t stream) {
    DeviceInfo di;
    obc_status st = device_info(&di);
    if (st != OBC_OK) return st;
    a.cap = (a.d + 3) & ~3;
    if (a.d > OBC_MAX_DCOL) return OBC_ERR_UNSUPPORTED;
    BlkPlan p;
    const int bc = (a.block_c == 4 || a.block_c == 8) ? a.block_c : 0;      // block pruning: the block size
    if (!blk_plan(a.d, a.w_trace != nullptr, di, &p, a.nm_prune > 0, bc, a.row_count, a.opts.threads)) return OBC_ERR_UNSUPPORTED;
    a.ms = p.ms;
    a.panel_floats = p.panel_floats;
    const int mp = a.opts.max_pending;
    a.max_pending = (mp >= 1 && mp <= BLK_MAXB) ? mp : BLK_MAXB;
    if (bc) {
        // the slots of a block must stay together: no on-chip tail (it compacts slot by slot), whole blocks per flush
        a.ms = 0;
        if (a.max_pending < bc) a.max_pending = bc;
        if (p.panel_floats / blk_ldz(a.cap) + p.g_vectors < bc) return OBC_ERR_UNSUPPORTED;
    }
    int blocks = di.sm_count * p.per_sm;
    if (a.row_count < blocks) blocks = a.row_count;
    a.Hws = nullptr;
    a.Gpan = nullptr;
    a.g_vectors = 0;
    a.g_ld = p.g_ld;
    a.ldp = a.cap;
    a.split = 0;
    a.split_state = nullptr; a.split_flags = nullptr; a.split_stride = 0;
    if (a.d > a.ms) {
        // Shares of rows (equal work per block instead of whole waves): when there are more rows than blocks and they
        // do not divide evenly; not with the N:M pattern or block pruning, whose extra per-row state is not handed over.
        // With one row per SM (long rows) at any number of waves: measured 5.2 waves of 3072-column rows 428 -> 385 ms,
        // 10.1 waves 794 -> 757 ms, 5.2 waves of 2304-column rows 219 -> 194 ms, of 1536-column rows 75.8 -> 68.7 ms.
        // With several rows per SM only up to three waves: the pieces are smaller and the kernels with this code slower,
        // above all the forced-order ones (10.4 waves of 768-column rows: trace 50.5 -> 51.0 ms, replay + quantisation
        // 51.1 -> 55.3 ms; 5.1 waves of 704-column rows 39.5 -> 40.5 and 42.5 -> 48.9 ms; 3.4 waves of 1408-column rows
        // gain, 79.9 -> 70.9 ms, 5.7 waves of 1152-column rows do not).
        const bool want_split = a.row_count > blocks && a.row_count % blocks != 0 && (p.per_sm == 1 || a.row_count < 3 * blocks) &&
                                a.nm_prune == 0 && !bc && !(a.opts.flags & OBC_ENGINE_WHOLE_WAVES);
        const size_t tri = round_up((size_t)blocks * (want_split ? 2 : 1) * a.d * a.cap * sizeof(float), 256);
        const size_t gpan = p.g_vectors ? round_up((size_t)blocks * p.g_vectors * p.g_ld * sizeof(float), 256) : 0;
        const size_t sst = want_split ? round_up((size_t)blocks * blk_split_stride(a.cap), 256) : 0;
        const size_t sfl = want_split ? round_up((size_t)blocks * sizeof(int), 256) : 0;
        if (!ws || !aligned256(ws) || ws_bytes < tri + gpan + sst + sfl) return OBC_ERR_WORKSPACE;
        a.Hws = reinterpret_cast<float*>(ws);
        if (p.g_vectors) {
            a.Gpan = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + tri);
            a.g_vectors = p.g_vectors;
        }
        if (want_split) {
            a.split = 1;
            a.split_state = reinterpret_cast<char*>(ws) + tri + gpan;
            a.split_stride = blk_split_stride(a.cap);
            a.split_flags = reinterpret_cast<int*>(reinterpret_cast<char*>(ws) + tri + gpan + sst);
        }
    }
    return blk_launch_nt(a, p.nt, blocks, p.smem, di.sm_count, stream);
}

obc_status blk_launch_nt(const EngineArgs& a, int nt, int blocks, size_t smem, int sm_count, cudaStream_t stream) {
    if (nt == 128) return blk_launch<128, 8>(a, blocks, smem, sm_count, stream);
    if (nt == 256) return blk_launch<256, 8>(a, blocks, smem, sm_count, stream);
    return blk_launch<512, 12>(a, blocks, smem, sm_count, stream);
}

}  // namespace obc
