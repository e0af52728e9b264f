// Tensor-core path of the layer Hessian H = 2 X X^T (Section 3 of "Optimal Brain Compression").
//
// A true dense contraction, so it runs on the 5th-generation tensor cores: TMA brings 128-row x 128-byte
// tiles of X (K-major for both operands) into 128B-swizzled shared memory, one elected thread issues
// tcgen05.mma with the FP32 accumulator in tensor memory, and four warps read the accumulator back with
// tcgen05.ld for the epilogue.  One CTA computes one 128 x 128 tile on or below the diagonal (SYRK) for one
// slice of the calibration axis; slices are combined in fixed order by the finalize kernel of hessian.cu.
//
// Two input precisions:
//   TF32    kind::tf32 reads the FP32 tiles as they are (10-bit mantissa per operand).
//   BF16X3  X is first split into hi = bf16(x) and lo = bf16(x - hi); the tile accumulates
//           hi*hi^T + hi*lo^T + lo*hi^T with kind::f16 (bf16 x bf16), which keeps ~16 mantissa bits.
//
// Every wait on an mbarrier is bounded (the limit of the pipeline's waits is a kernel argument).  If one expires,
// the CTA raises an error flag, waits -- with the full built-in limit -- for its own copies in flight and for the
// products it has issued, frees its tensor memory and returns; the finalize kernel then fills H with NaN and writes
// OBC_ERR_TIMEOUT to the caller's info word, so that the failure cannot go unnoticed downstream.
#include "common.cuh"
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>
#include <mutex>

namespace obc {

constexpr int TC_TILE = 128;          // output tile (M = N = 128)
constexpr int TC_KBYTES = 128;        // bytes of K per stage row = one 128B swizzle atom
constexpr int TC_THREADS = 128;
constexpr uint32_t TC_TILE_BYTES = TC_TILE * TC_KBYTES;      // 16 KiB per operand tile
constexpr int TC_WAIT_LIMIT = 4 * 1000 * 1000;      // polls of a bounded wait (about a second) unless the caller says otherwise

int hessian_splits(int d, int64_t n);
obc_status hessian_finalize_launch(const float* partial, int splits, int d, float* H, int ldh, int accumulate,
                                   const int* err, int32_t* info, cudaStream_t stream);

// ---- PTX wrappers ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait: false when the limit is reached
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int limit) {
    for (int i = 0; i < limit; ++i) {
        if (mbar_test(bar, parity)) return true;
        if (i > 64) __nanosleep(32);
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
template <int KIND>
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    if (KIND == 0)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile whose rows are 128 bytes, stored with the 128B
// swizzle (what TMA writes): 8-row groups are 1024 bytes apart, descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t dsc = 0;
    dsc |= (uint64_t)((addr >> 4) & 0x3fffu);          // start address, 16-byte units
    dsc |= (uint64_t)1 << 16;                           // leading byte offset (unused with swizzle): 1
    dsc |= (uint64_t)(1024 >> 4) << 32;                 // stride byte offset between 8-row groups
    dsc |= (uint64_t)1 << 46;                           // descriptor version (Blackwell)
    dsc |= (uint64_t)2 << 61;                           // SWIZZLE_128B
    return dsc;
}

// Instruction descriptor: FP32 accumulator, both operands K-major, M = N = 128.  fmt: 2 = TF32, 1 = BF16.
__host__ __device__ constexpr uint32_t instr_desc(uint32_t fmt) {
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(TC_TILE >> 3) << 17) | ((uint32_t)(TC_TILE >> 4) << 24);
}

// KIND 0: TF32, one tensor map per operand (FP32 data).  KIND 1: BF16X3, two maps per operand (hi, lo).
// CROSS = false: SYRK, both operands are row tiles of the same matrix (maps a == b), lower tile pairs only, d x d
// output.  CROSS = true: a general A B^T with A rows_a x n (maps a) and B rows_b x n (maps b), all tile pairs,
// rows_a x rows_b output (used for Y X^T of the dense refit).
template <int KIND, bool CROSS>
__global__ void __launch_bounds__(TC_THREADS) syrk_tc_kernel(const __grid_constant__ CUtensorMap map_a,
                                                             const __grid_constant__ CUtensorMap map_lo,
                                                             const __grid_constant__ CUtensorMap map_b,
                                                             const __grid_constant__ CUtensorMap map_blo,
                                                             int rows_a, int rows_b, int64_t n_elems, int64_t slice,
                                                             int stages, float* __restrict__ partial,
                                                             int* __restrict__ err, int wait_limit) {
    constexpr int TILES_PER_STAGE = KIND == 0 ? 2 : 4;             // A,B (+ A_lo, B_lo)
    constexpr int KELEMS = KIND == 0 ? 32 : 64;                    // elements of K per stage (128 bytes)
    constexpr int KSTEP = KIND == 0 ? 8 : 16;                      // elements of K per MMA (32 bytes)
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) unsigned long long bars[2 * 8 + 1];   // full[8], empty[8], accumulator-ready
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int mma_issued_s;                                   // the issuer has products in flight on the accumulator

    int bi = 0, bj = 0;
    if (CROSS) {
        const int tj = (rows_b + TC_TILE - 1) / TC_TILE;
        bi = blockIdx.x / tj; bj = blockIdx.x - bi * tj;
    } else {
        int t = blockIdx.x;
        while (t > bi) { t -= bi + 1; ++bi; }
        bj = t;
    }
    const int64_t kb0 = (int64_t)blockIdx.y * slice;
    const int64_t ke = kb0 + slice < n_elems ? kb0 + slice : n_elems;
    const int nkb = ke > kb0 ? (int)((ke - kb0 + KELEMS - 1) / KELEMS) : 0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[8]), accbar = smem_u32(&bars[16]);

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        mbar_init(accbar, 1);
        abort_s = 0;
        mma_issued_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {                                               // one warp allocates the accumulator columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(128));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_s;
    const uint32_t stage_bytes = TILES_PER_STAGE * TC_TILE_BYTES;
    int issued = 0;                                                // producer: k-blocks whose loads were issued

    if (warp == 0 && lane == 0) {
        // ---- TMA producer ---------------------------------------------------------------------------------
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % stages;
            if (kb >= stages && !mbar_wait(empty0 + 8 * s, ((kb / stages) - 1) & 1, wait_limit)) {
                atomicExch(err, 1); abort_s = 1; break;
            }
            if (*(volatile int*)&abort_s) break;
            const uint32_t dst = smem_u32(tiles) + s * stage_bytes;
            const int x = (int)(kb0 + (int64_t)kb * KELEMS);       // multiple of 128 bytes: satisfies the 16-byte rule
            mbar_expect_tx(full0 + 8 * s, stage_bytes);
            tma_load_2d(dst, &map_a, full0 + 8 * s, x, bi * TC_TILE);
            tma_load_2d(dst + TC_TILE_BYTES, &map_b, full0 + 8 * s, x, bj * TC_TILE);
            if (KIND == 1) {
                tma_load_2d(dst + 2 * TC_TILE_BYTES, &map_lo, full0 + 8 * s, x, bi * TC_TILE);
                tma_load_2d(dst + 3 * TC_TILE_BYTES, &map_blo, full0 + 8 * s, x, bj * TC_TILE);
            }
            issued = kb + 1;
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer -------------------------------------------------------------------------------------
        const uint32_t idesc = instr_desc(KIND == 0 ? 2u : 1u);
        for (int kb = 0; kb < nkb; ++kb) {
            const int s = kb % stages;
            if (!mbar_wait(full0 + 8 * s, (kb / stages) & 1, wait_limit)) { atomicExch(err, 2); abort_s = 1; break; }
            if (*(volatile int*)&abort_s) break;
            tc_fence_after();
            mma_issued_s = 1;
            const uint32_t base = smem_u32(tiles) + s * stage_bytes;
            const uint64_t da = smem_desc_sw128(base), db = smem_desc_sw128(base + TC_TILE_BYTES);
#pragma unroll
            for (int kk = 0; kk < KELEMS / KSTEP; ++kk) {
                const uint64_t adv = (uint64_t)(kk * 32 >> 4);     // 32 bytes of K per MMA, in 16-byte units
                const uint32_t acc = (kb > 0 || kk > 0) ? 1u : 0u;
                if (KIND == 0) {
                    tc_mma<0>(tmem_d, da + adv, db + adv, idesc, acc);
                } else {
                    const uint64_t dal = smem_desc_sw128(base + 2 * TC_TILE_BYTES), dbl = smem_desc_sw128(base + 3 * TC_TILE_BYTES);
                    tc_mma<1>(tmem_d, da + adv, db + adv, idesc, acc);        // hi * hi^T
                    tc_mma<1>(tmem_d, da + adv, dbl + adv, idesc, 1u);        // hi * lo^T
                    tc_mma<1>(tmem_d, dal + adv, db + adv, idesc, 1u);        // lo * hi^T
                }
            }
            tc_commit(empty0 + 8 * s);                             // frees the stage when these MMAs have read it
        }
        // accumulator complete (after an abort: completion of whatever was issued, which the exit path waits for)
        if (nkb > 0 && *(volatile int*)&mma_issued_s) tc_commit(accbar);
    }
    __syncwarp();
    // ---- epilogue: all four warps, warp w owns accumulator lanes 32w .. 32w+31 ------------------------------------
    bool ok = true;
    if (nkb > 0) {
        if (lane == 0) ok = mbar_wait(accbar, 0, wait_limit);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok && lane == 0) { atomicExch(err, 3); abort_s = 1; }
    }
    tc_fence_after();
    int ab = lane == 0 ? *(volatile int*)&abort_s : 0;
    ab = __shfl_sync(0xffffffffu, ab, 0);
    const bool aborted = !ok || ab != 0;                            // warp-uniform
    if (!aborted) {
        float* P = partial + (size_t)blockIdx.y * rows_a * rows_b;
        const int gi = bi * TC_TILE + warp * 32 + lane;
        for (int c = 0; c < TC_TILE / 32; ++c) {
            uint32_t r[32];
            if (nkb > 0) tmem_ld32(tmem_d + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c * 32), r);
            else {
#pragma unroll
                for (int q = 0; q < 32; ++q) r[q] = 0u;
            }
            if (gi < rows_a) {
                const int gj0 = bj * TC_TILE + c * 32;
#pragma unroll
                for (int q = 0; q < 32; ++q)
                    if (gj0 + q < rows_b) P[(size_t)gi * rows_b + gj0 + q] = __uint_as_float(r[q]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*(volatile int*)&abort_s && warp == 0 && lane == 0) {
        // Wait, with the full limit whatever the caller's, for our own copies in flight, so that nothing lands in
        // shared memory after we exit, and for the products issued so far, so that tensor memory is idle when it is
        // freed.  (Only the youngest phase of a stage can still be pending; older ones were consumed before reuse.)
        for (int kb = issued > stages ? issued - stages : 0; kb < issued; ++kb)
            mbar_wait(full0 + 8 * (kb % stages), (kb / stages) & 1, TC_WAIT_LIMIT);
        if (*(volatile int*)&mma_issued_s) mbar_wait(accbar, 0, TC_WAIT_LIMIT);
    }
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(128));
    }
}

// hi = bf16(x), lo = bf16(x - hi); outputs are d x n_pad (n_pad multiple of 64, padding written as zero)
__global__ void __launch_bounds__(256) split_bf16_kernel(const float* __restrict__ X, int d, int64_t n, int64_t ldx,
                                                         int64_t n_pad, __nv_bfloat16* __restrict__ hi,
                                                         __nv_bfloat16* __restrict__ lo) {
    const int64_t groups = n_pad / 8;
    const int64_t total = (int64_t)d * groups;
    for (int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; g < total; g += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = g / groups, k0 = (g % groups) * 8;
        float v[8];
        const float* src = X + row * ldx + k0;
        if (k0 + 7 < n) {
            const float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = (k0 + q < n) ? src[q] : 0.f;
        }
        __align__(16) __nv_bfloat16 h[8], l[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            h[q] = __float2bfloat16_rn(v[q]);
            l[q] = __float2bfloat16_rn(v[q] - __bfloat162float(h[q]));
        }
        *reinterpret_cast<uint4*>(hi + row * n_pad + k0) = *reinterpret_cast<const uint4*>(h);
        *reinterpret_cast<uint4*>(lo + row * n_pad + k0) = *reinterpret_cast<const uint4*>(l);
    }
}

// ---- host side ---------------------------------------------------------------------------------------------------
static PFN_cuTensorMapEncodeTiled encode_fn() {
    static std::mutex mu;
    static PFN_cuTensorMapEncodeTiled fn = nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(p);
    }
    return fn;
}

static bool make_map(CUtensorMap* map, CUtensorMapDataType type, int elem_bytes, const void* base, int64_t inner,
                     int64_t rows, int64_t row_stride_elems) {
    PFN_cuTensorMapEncodeTiled fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)row_stride_elems * elem_bytes};
    cuuint32_t box[2] = {(cuuint32_t)(TC_KBYTES / elem_bytes), (cuuint32_t)TC_TILE};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, type, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t hessian_tc_extra_bytes(int d, int64_t n) {          // error flag + bf16 hi/lo copies
    const int64_t n_pad = (n + 63) / 64 * 64;
    return 256 + 2 * round_up((size_t)d * n_pad * sizeof(__nv_bfloat16), 256);
}

// wait_limit: 0 = the built-in limit, > 0 = that many polls, < 0 = the pipeline's waits expire at once.
static int resolve_wait_limit(int wait_limit) { return wait_limit == 0 ? TC_WAIT_LIMIT : (wait_limit < 0 ? 0 : wait_limit); }

obc_status hessian_tc_launch(const float* X, int d, int64_t n, int64_t ldx, float* H, int ldh, int accumulate,
                             obc_prec prec, int32_t* info, int wait_limit, void* ws, cudaStream_t stream) {
    const int wl = resolve_wait_limit(wait_limit);
    const int splits = hessian_splits(d, n);
    char* p = reinterpret_cast<char*>(ws);
    float* partial = reinterpret_cast<float*>(p); p += round_up((size_t)splits * d * d * sizeof(float), 256);
    int* err = reinterpret_cast<int*>(p); p += 256;
    const int64_t n_pad = (n + 63) / 64 * 64;
    __nv_bfloat16* hi = reinterpret_cast<__nv_bfloat16*>(p); p += round_up((size_t)d * n_pad * sizeof(__nv_bfloat16), 256);
    __nv_bfloat16* lo = reinterpret_cast<__nv_bfloat16*>(p);
    OBC_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(int), stream));
    int64_t slice = (n + splits - 1) / splits;
    slice = (slice + 63) / 64 * 64;                          // whole 128-byte k-blocks in either precision
    const int T = (d + TC_TILE - 1) / TC_TILE;
    dim3 grid(T * (T + 1) / 2, splits);
    CUtensorMap ma, ml;
    if (prec == OBC_PREC_TF32) {
        if (!make_map(&ma, CU_TENSOR_MAP_DATA_TYPE_TFLOAT32, 4, X, n, d, ldx)) return OBC_ERR_CUDA;
        ml = ma;
        const int stages = 6;
        const size_t smem = (size_t)stages * 2 * TC_TILE_BYTES + 1024;
        OBC_CUDA_TRY(cudaFuncSetAttribute(syrk_tc_kernel<0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        syrk_tc_kernel<0, false><<<grid, TC_THREADS, smem, stream>>>(ma, ml, ma, ml, d, d, n, slice, stages, partial, err, wl);
        count_launch();
    } else {
        split_bf16_kernel<<<1184, 256, 0, stream>>>(X, d, n, ldx, n_pad, hi, lo);
        count_launch();
        if (!make_map(&ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, hi, n_pad, d, n_pad)) return OBC_ERR_CUDA;
        if (!make_map(&ml, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, lo, n_pad, d, n_pad)) return OBC_ERR_CUDA;
        const int stages = 3;
        const size_t smem = (size_t)stages * 4 * TC_TILE_BYTES + 1024;
        OBC_CUDA_TRY(cudaFuncSetAttribute(syrk_tc_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        syrk_tc_kernel<1, false><<<grid, TC_THREADS, smem, stream>>>(ma, ml, ma, ml, d, d, n_pad, slice, stages, partial, err, wl);
        count_launch();
    }
    OBC_CUDA_TRY(cudaGetLastError());
    return hessian_finalize_launch(partial, splits, d, H, ldh, accumulate, err, info, stream);
}

// ---- G (+)= alpha Y X^T on the tensor cores (appendix "Sequential Quantization with OBQ": X Y^T is accumulated over
// batches like the Hessian) ------------------------------------------------------------------------------------
int cross_splits(int rows_a, int rows_b, int64_t n) {
    const int tiles = ((rows_a + TC_TILE - 1) / TC_TILE) * ((rows_b + TC_TILE - 1) / TC_TILE);
    int64_t s = (444 + tiles - 1) / tiles;
    const int64_t by_len = (n + 2047) / 2048;
    if (by_len > s) s = by_len;
    if (s > 32) s = 32;
    if (s * 64 > n) s = n / 64;
    if (s < 1) s = 1;
    return (int)s;
}

size_t cross_workspace_bytes(int rows_a, int rows_b, int64_t n) {
    const int64_t n_pad = (n + 63) / 64 * 64;
    return round_up((size_t)cross_splits(rows_a, rows_b, n) * rows_a * rows_b * sizeof(float), 256) + 256 +
           2 * round_up((size_t)rows_a * n_pad * sizeof(__nv_bfloat16), 256) +
           2 * round_up((size_t)rows_b * n_pad * sizeof(__nv_bfloat16), 256);
}

__global__ void __launch_bounds__(256) cross_finalize_kernel(const float* __restrict__ partial, int splits, int rows_a,
                                                             int rows_b, float* __restrict__ G, int ldg, int accumulate,
                                                             float alpha, const int* __restrict__ err,
                                                             int32_t* __restrict__ info) {
    const int i = blockIdx.y;
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (info && i == 0 && j == 0) info[0] = (err && *err != 0) ? (int32_t)OBC_ERR_TIMEOUT : 0;
    if (j >= rows_b) return;
    float s = 0.f;
    for (int z = 0; z < splits; ++z) s += partial[(size_t)z * rows_a * rows_b + (size_t)i * rows_b + j];
    s *= alpha;
    if (accumulate) s += G[(size_t)i * ldg + j];
    if (err && *err != 0) s = __int_as_float(0x7fc00000);
    G[(size_t)i * ldg + j] = s;
}

obc_status cross_tc_launch(const float* Y, int rows_a, int64_t ldy, const float* X, int rows_b, int64_t ldx, int64_t n,
                           float* G, int ldg, int accumulate, float alpha, obc_prec prec, int32_t* info, int wait_limit,
                           void* ws, cudaStream_t stream) {
    const int wl = resolve_wait_limit(wait_limit);
    const int splits = cross_splits(rows_a, rows_b, n);
    char* p = reinterpret_cast<char*>(ws);
    float* partial = reinterpret_cast<float*>(p); p += round_up((size_t)splits * rows_a * rows_b * sizeof(float), 256);
    int* err = reinterpret_cast<int*>(p); p += 256;
    const int64_t n_pad = (n + 63) / 64 * 64;
    __nv_bfloat16* yhi = reinterpret_cast<__nv_bfloat16*>(p); p += round_up((size_t)rows_a * n_pad * sizeof(__nv_bfloat16), 256);
    __nv_bfloat16* ylo = reinterpret_cast<__nv_bfloat16*>(p); p += round_up((size_t)rows_a * n_pad * sizeof(__nv_bfloat16), 256);
    __nv_bfloat16* xhi = reinterpret_cast<__nv_bfloat16*>(p); p += round_up((size_t)rows_b * n_pad * sizeof(__nv_bfloat16), 256);
    __nv_bfloat16* xlo = reinterpret_cast<__nv_bfloat16*>(p);
    OBC_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(int), stream));
    int64_t slice = (n + splits - 1) / splits;
    slice = (slice + 63) / 64 * 64;
    const int ti = (rows_a + TC_TILE - 1) / TC_TILE, tj = (rows_b + TC_TILE - 1) / TC_TILE;
    dim3 grid(ti * tj, splits);
    CUtensorMap ma, mal, mb, mbl;
    if (prec == OBC_PREC_TF32) {
        if (!make_map(&ma, CU_TENSOR_MAP_DATA_TYPE_TFLOAT32, 4, Y, n, rows_a, ldy)) return OBC_ERR_CUDA;
        if (!make_map(&mb, CU_TENSOR_MAP_DATA_TYPE_TFLOAT32, 4, X, n, rows_b, ldx)) return OBC_ERR_CUDA;
        mal = ma; mbl = mb;
        const int stages = 6;
        const size_t smem = (size_t)stages * 2 * TC_TILE_BYTES + 1024;
        OBC_CUDA_TRY(cudaFuncSetAttribute(syrk_tc_kernel<0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        syrk_tc_kernel<0, true><<<grid, TC_THREADS, smem, stream>>>(ma, mal, mb, mbl, rows_a, rows_b, n, slice, stages, partial, err, wl);
        count_launch();
    } else {
        split_bf16_kernel<<<1184, 256, 0, stream>>>(Y, rows_a, n, ldy, n_pad, yhi, ylo);
        split_bf16_kernel<<<1184, 256, 0, stream>>>(X, rows_b, n, ldx, n_pad, xhi, xlo);
        count_launch(2);
        if (!make_map(&ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, yhi, n_pad, rows_a, n_pad)) return OBC_ERR_CUDA;
        if (!make_map(&mal, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ylo, n_pad, rows_a, n_pad)) return OBC_ERR_CUDA;
        if (!make_map(&mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, xhi, n_pad, rows_b, n_pad)) return OBC_ERR_CUDA;
        if (!make_map(&mbl, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, xlo, n_pad, rows_b, n_pad)) return OBC_ERR_CUDA;
        const int stages = 3;
        const size_t smem = (size_t)stages * 4 * TC_TILE_BYTES + 1024;
        OBC_CUDA_TRY(cudaFuncSetAttribute(syrk_tc_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        syrk_tc_kernel<1, true><<<grid, TC_THREADS, smem, stream>>>(ma, mal, mb, mbl, rows_a, rows_b, n_pad, slice, stages, partial, err, wl);
        count_launch();
    }
    OBC_CUDA_TRY(cudaGetLastError());
    dim3 fgrid((rows_b + 255) / 256, rows_a);
    cross_finalize_kernel<<<fgrid, 256, 0, stream>>>(partial, splits, rows_a, rows_b, G, ldg, accumulate, alpha, err, info);
    count_launch();
    OBC_CUDA_TRY(cudaGetLastError());
    return OBC_OK;
}

}  // namespace obc
