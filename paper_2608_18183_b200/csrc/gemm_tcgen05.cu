// bf16 decoder GEMM on the 5th-generation tensor cores: C[M,N] fp32 (+)= A[M,K] . W[N,K]^T.
//
// Both operands are K-major (activations row-major [M,K], weights row-major [N,K]), so each CTA
// streams 128 x 64 (A) and BN x 64 (W) bf16 tiles through a TMA -> shared-memory ring
// (128-byte swizzle), one elected thread issues tcgen05.mma (M=128, N=BN, K=16) into a TMEM
// accumulator, and four warps read the accumulator back with tcgen05.ld for the epilogue.
// The K loop is fixed (no split-K), so an output element's rounding does not depend on M or on
// which rows share its tile: Full and Compact execution give identical bits.
//
// Every mbarrier wait is bounded: after the limit the kernel raises the error flag, drains, frees its
// TMEM and returns.  No cluster launch, no multicast.
#include <cuda.h>

#include <cstdio>

#include "internal.h"

namespace hbsjd {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;  // 64 bf16 = 128 bytes = one swizzle row

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait (about one second).  Returns false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
        for (int it = 0; it < 256; ++it)
            if (mbar_try(bar, parity)) return true;
        if (globaltimer_ns() - t0 > 1000000000ull) return false;
    }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    d |= (uint64_t)1 << 16;                        // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                        // 128-byte swizzle
    return d;
}

// Instruction descriptor: D fp32, A/B bf16, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t umma_idesc(int bn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <int BN>
struct Cfg {
    static constexpr int STAGES = BN >= 256 ? 4 : (BN == 128 ? 3 : 4);
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int TMEM_COLS = BN < 32 ? 32 : BN;
    static constexpr int SMEM = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int BN>
__global__ void __launch_bounds__(128) k_gemm_tcgen05(const __grid_constant__ CUtensorMap map_a,
                                                      const __grid_constant__ CUtensorMap map_w,
                                                      float* __restrict__ C, int M, int N, int K, int accumulate,
                                                      int32_t* __restrict__ error_flag) {
    using cfg = Cfg<BN>;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;            // 1024-byte aligned tile ring
    const uint32_t bars = tiles + cfg::STAGES * cfg::STAGE_BYTES;  // full[STAGES], empty[STAGES], accum, tmem slot
    unsigned char* bars_ptr = smem_raw + (bars - raw);
    const uint32_t full0 = bars, empty0 = bars + 8 * cfg::STAGES, accum_bar = bars + 16 * cfg::STAGES;
    volatile uint32_t* tmem_slot = (volatile uint32_t*)(bars_ptr + 16 * cfg::STAGES + 8);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, m0 = blockIdx.y * BM;
    const int num_kb = K / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < cfg::STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        mbar_init(accum_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                         smem_u32((const void*)tmem_slot)),
                     "r"((uint32_t)cfg::TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0 && lane == 0) {
        // ---- TMA producer
        for (int kb = 0; kb < num_kb; ++kb) {
            const int s = kb % cfg::STAGES;
            if (kb >= cfg::STAGES) {
                if (!mbar_wait(empty0 + 8 * s, ((kb / cfg::STAGES) - 1) & 1)) {
                    *abort_flag = 1;
                    atomicExch(error_flag, 1);
                    break;
                }
            }
            const uint32_t a_dst = tiles + s * cfg::STAGE_BYTES;
            const uint32_t b_dst = a_dst + cfg::A_BYTES;
            mbar_expect_tx(full0 + 8 * s, cfg::STAGE_BYTES);
            tma_load_2d(a_dst, &map_a, kb * BK, m0, full0 + 8 * s);
            tma_load_2d(b_dst, &map_w, kb * BK, n0, full0 + 8 * s);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer
        constexpr uint32_t idesc = umma_idesc(BN);
        bool ok = true;
        for (int kb = 0; kb < num_kb && ok; ++kb) {
            const int s = kb % cfg::STAGES;
            if (!mbar_wait(full0 + 8 * s, (kb / cfg::STAGES) & 1)) {
                *abort_flag = 1;
                atomicExch(error_flag, 2);
                ok = false;
                break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_src = tiles + s * cfg::STAGE_BYTES;
            const uint32_t b_src = a_src + cfg::A_BYTES;
#pragma unroll
            for (int k = 0; k < BK / 16; ++k) {
                const uint64_t da = umma_desc(a_src + k * 32);
                const uint64_t db = umma_desc(b_src + k * 32);
                umma_f16(tmem_base, da, db, idesc, (kb | k) != 0 ? 1u : 0u);
            }
            umma_commit(empty0 + 8 * s);  // frees the stage once these MMAs have read it
        }
        umma_commit(accum_bar);  // accumulator complete (also arrives on the abort path)
    }
    __syncwarp();

    // ---- epilogue: all four warps; warp w owns TMEM lanes 32w..32w+31 = tile rows 32w..32w+31
    const bool ready = mbar_wait(accum_bar, 0);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (!ready && lane == 0) atomicExch(error_flag, 3);
    const bool good = ready && (*abort_flag == 0);
    const int row = m0 + warp * 32 + lane;
    if (good) {
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
            uint32_t r[32];
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0;
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                  "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
                  "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
                  "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
                  "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                : "r"(taddr)
                : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (row < M) {
                float4* dst = reinterpret_cast<float4*>(C + (size_t)row * N + n0 + c0);
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    float4 o = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                           __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                    if (accumulate) {
                        const float4 old = dst[v];
                        o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                    }
                    dst[v] = o;
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                     "r"((uint32_t)cfg::TMEM_COLS)
                     : "memory");
    }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                             const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
    static EncodeFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeFn)p;
    }
    return fn;
}

// 2D bf16 row-major [rows, K] tensor, box = [box_rows, 64], 128-byte swizzle, zero fill out of bounds.
bool make_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
    EncodeFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
cudaError_t launch(const CUtensorMap& ma, const CUtensorMap& mw, float* C, int M, int N, int K, int accumulate,
                   int32_t* error_flag, cudaStream_t s) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(k_gemm_tcgen05<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg<BN>::SMEM);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid(N / BN, (M + BM - 1) / BM);
    k_gemm_tcgen05<BN><<<grid, 128, Cfg<BN>::SMEM, s>>>(ma, mw, C, M, N, K, accumulate, error_flag);
    return cudaGetLastError();
}

}  // namespace

int gemm_tcgen05_tile_n(int M, int N) {
    const long tiles_m = (M + BM - 1) / BM;
    if (N % 128 == 0 && tiles_m * (N / 128) >= 2 * 148) return 128;
    if (N % 64 == 0 && tiles_m * (N / 64) >= 148) return 64;
    if (N % 32 == 0) return 32;
    return 64;
}

int gemm_tcgen05_run(const bf16* A, const bf16* W, float* C, int M, int N, int K, int accumulate, int force_bn,
                     int32_t* error_flag, cudaStream_t s, char* err, size_t errlen) {
    if (M <= 0) return 0;
    if (K % BK != 0 || N % 32 != 0 || (((uintptr_t)A | (uintptr_t)W | (uintptr_t)C) & 15)) {
        snprintf(err, errlen, "gemm: needs K %% 64 == 0, N %% 32 == 0 and 16-byte aligned operands (M=%d N=%d K=%d)",
                 M, N, K);
        return -1;
    }
    const int bn = force_bn ? force_bn : gemm_tcgen05_tile_n(M, N);
    if (N % bn != 0) {
        snprintf(err, errlen, "gemm: N=%d is not a multiple of the tile width %d", N, bn);
        return -1;
    }
    CUtensorMap ma, mw;
    if (!make_map(&ma, A, M, K, BM) || !make_map(&mw, W, N, K, bn)) {
        snprintf(err, errlen, "gemm: cuTensorMapEncodeTiled failed (M=%d N=%d K=%d)", M, N, K);
        return -3;
    }
    cudaError_t e;
    switch (bn) {
        case 32: e = launch<32>(ma, mw, C, M, N, K, accumulate, error_flag, s); break;
        case 64: e = launch<64>(ma, mw, C, M, N, K, accumulate, error_flag, s); break;
        case 128: e = launch<128>(ma, mw, C, M, N, K, accumulate, error_flag, s); break;
        case 256: e = launch<256>(ma, mw, C, M, N, K, accumulate, error_flag, s); break;
        default: snprintf(err, errlen, "gemm: unsupported tile width %d", bn); return -1;
    }
    if (e != cudaSuccess) {
        snprintf(err, errlen, "gemm launch: %s", cudaGetErrorString(e));
        return -3;
    }
    return 0;
}

}  // namespace hbsjd
