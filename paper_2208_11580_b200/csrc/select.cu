// Global mask selection (Algorithm 2 of "Optimal Brain Compression", appendix "ExactOBS Global Step").
//
// The sequential procedure pops, k times, the row whose NEXT recorded loss is smallest (ties: lowest row).
// A row's losses need not be monotone, so a cheap entry hidden behind an expensive one is only reached
// after the expensive one was popped.  Equivalent parallel form: give entry (r,t) the key
// max_{t'<=t} L[r][t'] (prefix maximum); the procedure then pops exactly the k smallest entries in the
// lexicographic order (key, r, t).  Within a row keys are non-decreasing, so the popped entries of a row
// are a prefix and counts[r] = #{key < T} + (share of the entries with key == T, handed out by row).
//
// Kernels: prefix-max keys -> 4-pass 8-bit radix select of the k-th key T -> per-row counts -> tie
// distribution over rows -> mask scatter.  Keys are non-negative floats compared as unsigned integers.
#include "common.cuh"
#include <mutex>

namespace obc {

constexpr int SEL_THREADS = 256;

struct SelectState {            // lives in the workspace
    unsigned int hist[256];
    unsigned int prefix;        // bits of T decided so far
    unsigned int pad;
    unsigned long long remaining;   // rank still to resolve inside the current prefix bucket (1-based)
};

__device__ __forceinline__ unsigned int loss_key(float x) {
    // losses are >= 0; NaN and negative values are mapped to the ends so that the order stays total
    if (x != x) return 0x7f800000u;          // NaN -> +inf
    if (x <= 0.f) return 0u;                 // -0, negatives
    return __float_as_uint(x);
}

// keys[r][t] = max_{t' <= t} key(L[r][t'])       one block per row
__global__ void __launch_bounds__(SEL_THREADS) prefix_max_kernel(const float* __restrict__ loss, int d,
                                                                 unsigned int* __restrict__ keys) {
    __shared__ unsigned int part[SEL_THREADS];
    const int r = blockIdx.x, tid = threadIdx.x;
    const int chunk = (d + SEL_THREADS - 1) / SEL_THREADS;
    const int b = tid * chunk, e = min(d, b + chunk);
    const float* L = loss + (size_t)r * d;
    unsigned int* K = keys + (size_t)r * d;
    unsigned int mx = 0;
    for (int t = b; t < e; ++t) mx = max(mx, loss_key(L[t]));
    part[tid] = mx;
    __syncthreads();
    for (int off = 1; off < SEL_THREADS; off <<= 1) {           // inclusive max-scan of the chunk maxima
        unsigned int o = tid >= off ? part[tid - off] : 0u;
        __syncthreads();
        part[tid] = max(part[tid], o);
        __syncthreads();
    }
    unsigned int run = tid ? part[tid - 1] : 0u;
    for (int t = b; t < e; ++t) { run = max(run, loss_key(L[t])); K[t] = run; }
}

__global__ void select_init_kernel(SelectState* s, long long k) {
    if (threadIdx.x < 256) s->hist[threadIdx.x] = 0;
    if (threadIdx.x == 0) { s->prefix = 0; s->remaining = (unsigned long long)k; }
}

// histogram of the digit at `shift` over keys whose higher bits equal the decided prefix
__global__ void __launch_bounds__(SEL_THREADS) select_hist_kernel(const unsigned int* __restrict__ keys, long long n,
                                                                  int shift, SelectState* s) {
    __shared__ unsigned int h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const unsigned int prefix = s->prefix;
    const unsigned int himask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
    for (long long i = blockIdx.x * (long long)SEL_THREADS + threadIdx.x; i < n; i += (long long)gridDim.x * SEL_THREADS) {
        const unsigned int key = keys[i];
        if ((key & himask) == prefix) atomicAdd(&h[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (h[threadIdx.x]) atomicAdd(&s->hist[threadIdx.x], h[threadIdx.x]);
}

// pick the digit that contains rank `remaining`, update prefix / remaining, clear the histogram
__global__ void select_pick_kernel(SelectState* s, int shift) {
    if (threadIdx.x == 0) {
        unsigned long long rem = s->remaining, acc = 0;
        int dgt = 255;
        if (rem == 0) { dgt = 0; }      // k == 0: T = 0 with nothing to take
        else {
            for (int b = 0; b < 256; ++b) {
                const unsigned long long c = s->hist[b];
                if (acc + c >= rem) { dgt = b; break; }
                acc += c;
            }
            rem -= acc;
        }
        s->prefix |= ((unsigned int)dgt) << shift;
        s->remaining = rem;
    }
    __syncthreads();
    if (threadIdx.x < 256) s->hist[threadIdx.x] = 0;
}

// per row: how many keys are below T, how many equal T          one block per row
__global__ void __launch_bounds__(SEL_THREADS) select_count_kernel(const unsigned int* __restrict__ keys, int d,
                                                                   const SelectState* s, int* __restrict__ lt,
                                                                   int* __restrict__ eq) {
    __shared__ int sl[SEL_THREADS], se[SEL_THREADS];
    const unsigned int T = s->prefix;
    const unsigned int* K = keys + (size_t)blockIdx.x * d;
    int l = 0, e = 0;
    for (int t = threadIdx.x; t < d; t += SEL_THREADS) { const unsigned int k = K[t]; l += k < T; e += k == T; }
    sl[threadIdx.x] = l; se[threadIdx.x] = e;
    __syncthreads();
    for (int off = SEL_THREADS / 2; off; off >>= 1) {
        if (threadIdx.x < off) { sl[threadIdx.x] += sl[threadIdx.x + off]; se[threadIdx.x] += se[threadIdx.x + off]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) { lt[blockIdx.x] = sl[0]; eq[blockIdx.x] = se[0]; }
}

// hand the `remaining` entries with key == T to the rows in row order      single block
__global__ void __launch_bounds__(SEL_THREADS) select_ties_kernel(const SelectState* s, const int* __restrict__ lt,
                                                                  const int* __restrict__ eq, int rows,
                                                                  int* __restrict__ counts) {
    __shared__ unsigned long long part[SEL_THREADS];
    const int tid = threadIdx.x;
    const int chunk = (rows + SEL_THREADS - 1) / SEL_THREADS;
    const int b = tid * chunk, e = min(rows, b + chunk);
    unsigned long long sum = 0;
    for (int r = b; r < e; ++r) sum += (unsigned long long)eq[r];
    part[tid] = sum;
    __syncthreads();
    if (tid == 0) {
        unsigned long long acc = 0;
        for (int i = 0; i < SEL_THREADS; ++i) { const unsigned long long c = part[i]; part[i] = acc; acc += c; }
    }
    __syncthreads();
    unsigned long long before = part[tid];
    const unsigned long long rem = s->remaining;
    for (int r = b; r < e; ++r) {
        const unsigned long long c = (unsigned long long)eq[r];
        unsigned long long take = rem > before ? rem - before : 0ull;
        if (take > c) take = c;
        counts[r] = lt[r] + (int)take;
        before += c;
    }
}

// mask[r][:] = 1, then 0 at the first counts[r] entries of the row's order     one block per row
__global__ void __launch_bounds__(SEL_THREADS) mask_kernel(const int32_t* __restrict__ order, const int* __restrict__ counts,
                                                           int d, uint8_t* __restrict__ mask) {
    const int r = blockIdx.x;
    uint8_t* M = mask + (size_t)r * d;
    for (int j = threadIdx.x; j < d; j += SEL_THREADS) M[j] = 1;
    __syncthreads();
    const int c = min(counts[r], d);
    for (int t = threadIdx.x; t < c; t += SEL_THREADS) {
        const int j = order[(size_t)r * d + t];
        if (j >= 0 && j < d) M[j] = 0;
    }
}

size_t select_workspace_bytes(int rows, int d) {
    return round_up((size_t)rows * d * 4, 256) + round_up(sizeof(SelectState), 256) + 2 * round_up((size_t)rows * 4, 256);
}

obc_status select_launch(const float* loss, const int32_t* order, int rows, int d, int64_t k, int32_t* counts,
                         uint8_t* mask, void* ws, cudaStream_t stream) {
    char* p = reinterpret_cast<char*>(ws);
    unsigned int* keys = reinterpret_cast<unsigned int*>(p); p += round_up((size_t)rows * d * 4, 256);
    SelectState* st = reinterpret_cast<SelectState*>(p); p += round_up(sizeof(SelectState), 256);
    int* lt = reinterpret_cast<int*>(p); p += round_up((size_t)rows * 4, 256);
    int* eq = reinterpret_cast<int*>(p);
    const long long n = (long long)rows * d;
    prefix_max_kernel<<<rows, SEL_THREADS, 0, stream>>>(loss, d, keys);
    count_launch();
    select_init_kernel<<<1, 256, 0, stream>>>(st, (long long)k);
    count_launch();
    int hb = (int)((n + SEL_THREADS * 8 - 1) / (SEL_THREADS * 8));
    if (hb > 1184) hb = 1184;
    if (hb < 1) hb = 1;
    for (int shift = 24; shift >= 0; shift -= 8) {
        select_hist_kernel<<<hb, SEL_THREADS, 0, stream>>>(keys, n, shift, st);
        count_launch();
        select_pick_kernel<<<1, 256, 0, stream>>>(st, shift);
        count_launch();
    }
    select_count_kernel<<<rows, SEL_THREADS, 0, stream>>>(keys, d, st, lt, eq);
    count_launch();
    select_ties_kernel<<<1, SEL_THREADS, 0, stream>>>(st, lt, eq, rows, counts);
    count_launch();
    mask_kernel<<<rows, SEL_THREADS, 0, stream>>>(order, counts, d, mask);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

// ---- allocation-free variant ----------------------------------------------------------------------------------
// Scratch for obc_select_global_mask_static: a fixed array in device memory that every GPU loading this library
// holds until the process exits.  Sized for OBC_SELECT_STATIC_MAX_KEYS loss entries and
// OBC_SELECT_STATIC_MAX_ROWS rows (16 MiB of keys + 128 KiB of per-row counters + the selection state).
constexpr size_t SELECT_STATIC_BYTES =
    ((size_t)OBC_SELECT_STATIC_MAX_KEYS * 4 + 255) / 256 * 256 + (sizeof(SelectState) + 255) / 256 * 256 +
    2 * (((size_t)OBC_SELECT_STATIC_MAX_ROWS * 4 + 255) / 256 * 256);
static __device__ __align__(256) unsigned char g_select_scratch[SELECT_STATIC_BYTES];

// Device address of the array on the CURRENT device.  In host code the array's name is only a stand-in, so
// the address is looked up once per device (with that device current) and cached.
static obc_status select_static_scratch(void** out) {
    static std::mutex mu;
    static void* ptrs[64] = {};
    int dev = 0;
    OBC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return OBC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        OBC_CUDA_TRY(cudaGetSymbolAddress(&p, g_select_scratch));
        if (!p) return OBC_ERR_CUDA;
        ptrs[dev] = p;
    }
    *out = ptrs[dev];
    return OBC_OK;
}

}  // namespace obc

extern "C" obc_status obc_select_global_mask_static(const float* loss, const int32_t* order, int d_row, int d_col,
                                                    int64_t k, int32_t* counts, uint8_t* mask, obc_stream stream) {
    using namespace obc;
    if (d_row <= 0 || d_col <= 0 || !loss || !order || !counts || !mask) return OBC_ERR_INVALID_ARG;
    if (k < 0 || k > (int64_t)d_row * d_col) return OBC_ERR_INVALID_ARG;
    if (d_row > OBC_SELECT_STATIC_MAX_ROWS || (int64_t)d_row * d_col > (int64_t)OBC_SELECT_STATIC_MAX_KEYS)
        return OBC_ERR_STATIC_SCRATCH;
    void* scratch = nullptr;
    const obc_status st = select_static_scratch(&scratch);
    if (st != OBC_OK) return st;
    // every launch sequence re-initialises the selection state and overwrites the keys / counters it reads
    return select_launch(loss, order, d_row, d_col, k, counts, mask, scratch, (cudaStream_t)stream);
}
