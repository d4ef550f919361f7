// bf16 decoder GEMMs on the 5th-generation tensor cores: acc[M,N] = A[M,K] . W[N,K]^T with fused epilogues.
//
// Both operands are K-major (activations row-major [M,K], weights row-major [N,K]).  The kernel is
// persistent and warp-specialised: one CTA (or CTA pair) per SM walks a static list of 128 x BN output tiles;
//   warp 0 (one lane)  TMA producer: 128 x 64 (A) and BN x 64 (W) bf16 tiles, 128-byte swizzle, STAGES-deep ring
//   warp 1 (one lane)  issues tcgen05.mma (M = 128, N = BN, K = 16) into one of two TMEM accumulators
//   warps 2..5         epilogue: tcgen05.ld of the finished accumulator while the next tile's main loop runs
// BN = 256 keeps the shared-memory operand traffic per MMA below the 128 B/clk the SM can supply.
// The K loop is fixed (no split-K), so an output element's rounding does not depend on M or on which rows
// share its tile: Full and Compact execution give identical bits.
//
// Epilogues:  STORE  C fp32 = acc           (LM head -> logits)
//             ADD    C fp32 += acc          (public hbsjd_gemm with accumulate)
//             ADDNORM  C fp32 += acc, bf16 copy of the new C, per-row partial sums of squares   (attention-out and
//                    FFN-down projections into the residual stream; feeds the RMSNorm folded into the next GEMM)
//             SWIGLU out bf16[M, N/2] = silu(acc[2f]) * acc[2f+1]   (gate/up rows interleaved at load time)
//             QKV    2D RoPE on q and k, bf16 q[M, D], k and v written to the row's KV pages
//
// Large problems run 256 x 256 tiles on CTA pairs (clusters of two, cta_group::2 MMAs; see Cfg below).  The
// weight tiles of a CTA's first ring revolution are requested before the grid dependency resolves.
//
// Every mbarrier wait is bounded (about a second): after the limit the kernel raises the error flag, all
// roles leave their loops, TMEM is freed and the kernel returns.  No multicast loads anywhere (the only
// multicast is tcgen05.commit arriving on both CTAs of a pair).
#include <cuda.h>

#include <cstdio>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <functional>
#include <mutex>
#include <unordered_map>

#include "internal.h"

namespace hbsjd {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;  // 64 bf16 = 128 bytes = one swizzle row
constexpr int NUM_THREADS = 192;

enum { EPI_STORE = 0, EPI_ADD = 1, EPI_SWIGLU = 2, EPI_QKV = 3, EPI_ADDNORM = 4 };

struct GemmArgs {
    float* C;        // STORE / ADD
    bf16* out;       // SWIGLU: [M, N/2];  QKV: q [M, D]
    int M, N, K;
    int32_t* error_flag;
    // RMSNorm folded around the GEMMs (bf16 model): the operand A is the bf16 copy of the UNNORMALISED residual
    // stream and the norm's gain is folded into W, so that norm(x) W^T = r (x W'^T) with the row factor
    // r = rsqrt(mean(x^2) + eps) applied here, in the epilogue, from partial sums of squares
    const float* ssq_in;   // [M][ssq_n] partial sums of squares of A's rows (null: no row factor)
    int ssq_n;             // partials per row = K / 32
    float inv_dim, eps;
    // ADDNORM: C (fp32 residual) += acc, plus what the next GEMM needs
    bf16* hb;              // [M][N] bf16 copy of the updated residual
    float* ssq_out;        // [M][N / 32] sums of squares of the updated residual per 32-column chunk
    int w_constant;   // W never changes while the stream runs (model weights): its tiles may be fetched early
    unsigned int acc_wait_ns;  // 0, or a shorter limit for the epilogue's accumulator wait (time-out test)
    // QKV epilogue
    State st;
    int S, layer;
    const float* rope_cs;  // [T][dh/2][2]
    KvView kv;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// Bounded wait (about one second unless a shorter limit is given).  Returns false when it gave up or another
// role raised `abort`.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort,
                                          unsigned long long limit_ns = 1000000000ull) {
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    const int polls = limit_ns < 1000000ull ? 1 : 128;  // a short limit is checked after every poll
    for (;;) {
        for (int it = 0; it < polls; ++it)
            if (mbar_try(bar, parity)) return true;
        if (*abort) return false;
        if (globaltimer_ns() - t0 > limit_ns) return false;
    }
}


__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// CTA-pair variants (cta_group::2): the load may signal the mbarrier of the pair's leader.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Raises the CTA's abort flag and, in a CTA pair, the partner's, so that neither spends its own time-outs.
template <bool PAIR>
__device__ __forceinline__ void raise_abort(volatile uint32_t* abort_flag, uint32_t rank) {
    *abort_flag = 1;
    if (PAIR) {
        const uint32_t remote = map_to_rank(smem_u32((const void*)abort_flag), rank ^ 1u);
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(remote), "r"(1u) : "memory");
    }
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(acc)
        : "memory");
}
// arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair once the MMAs issued so far
// have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
        "h"((unsigned short)3)
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
__host__ __device__ constexpr uint32_t umma_idesc(int bn, int bm = BM) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(bm >> 4) << 24);
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
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t r[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// PAIR: two CTAs of a cluster compute one 256 x BN tile with cta_group::2 MMAs; each CTA stages its own 128 rows
// of A and its own BN/2 rows of W, which cuts the operand bytes per FLOP by a third against a 128 x BN tile.
// WIDE: the epilogue stages a bf16 tile beside every fp32 tile (EPI_ADDNORM), 48 KB instead of 32 KB; the operand
// ring gives up a stage or two for it.
template <int BN, bool PAIR = false, bool WIDE = false>
struct Cfg {
    // as many stages as fit beside the epilogue staging: small tiles are latency-bound (one TMA round trip per ring
    // revolution), so a narrow tile gets a deep ring
    static constexpr int STAGES = WIDE ? (PAIR ? 5 : (BN >= 256 ? 3 : (BN == 128 ? 5 : (BN == 64 ? 6 : 8))))
                                       : (PAIR ? 6 : (BN >= 256 ? 4 : (BN == 128 ? 6 : 8)));
    // k-blocks that share one full / empty barrier pair (one wait and one commit per KG x 4 MMAs)
    static constexpr int KG = WIDE ? ((PAIR || BN >= 128) ? 1 : (BN == 64 ? 2 : 4)) : ((!PAIR && BN <= 64) ? 4 : 2);
    static constexpr int GROUPS = STAGES / KG;
    static_assert(GROUPS * KG == STAGES && GROUPS >= 2, "ring stages must split into whole barrier groups");
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int B_BYTES = (PAIR ? BN / 2 : BN) * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;  // two accumulators
    // 4 epilogue warps x 2 buffers x (32 rows x 128 bytes fp32 [+ 32 rows x 64 bytes bf16])
    static constexpr int WARP_STAGING = WIDE ? 2 * 6144 : 2 * 4096;
    static constexpr int STAGING_BYTES = 4 * WARP_STAGING;
    static constexpr int SMEM = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
    static_assert(16 * STAGES + 32 + 8 + 8 <= 256, "barrier area");
    static_assert(SMEM <= 227 * 1024, "shared memory of one CTA");
};

// Per-row context of the QKV epilogue: where the token row's q / k / v go.
struct RowDst {
    bool valid;
    int s;        // sequence index (RoPE position)
    size_t kvoff; // element offset of the row's K/V vector in the page pool
};

template <int BN, int EPI, bool PAIR>
__global__ void __launch_bounds__(NUM_THREADS) k_gemm_tcgen05(const __grid_constant__ CUtensorMap map_a,
                                                              const __grid_constant__ CUtensorMap map_w,
                                                              const __grid_constant__ CUtensorMap map_c,
                                                              const __grid_constant__ CUtensorMap map_hb,
                                                              const GemmArgs g) {
    using cfg = Cfg<BN, PAIR, EPI == EPI_ADDNORM>;
    extern __shared__ unsigned char smem_raw[];
    pdl_trigger();
    const uint32_t rank = PAIR ? cluster_rank() : 0u;       // 0 = leader of the pair
    const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;  // tile walker id
    const int units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    constexpr int TM = PAIR ? 2 * BM : BM;                  // tile rows
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;  // 1024-byte aligned tile ring
    const uint32_t staging = tiles + cfg::STAGES * cfg::STAGE_BYTES;  // 1024-byte aligned
    const uint32_t bars = staging + cfg::STAGING_BYTES;
    unsigned char* bars_ptr = smem_raw + (bars - raw);
    // full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], tmem slot, abort flag
    const uint32_t full0 = bars, empty0 = bars + 8 * cfg::STAGES;
    const uint32_t accf0 = bars + 16 * cfg::STAGES, acce0 = accf0 + 16;
    volatile uint32_t* tmem_slot = (volatile uint32_t*)(bars_ptr + 16 * cfg::STAGES + 32);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    const uint32_t drain_bar = acce0 + 16 + 8;  // behind the tmem slot and the abort flag: used on the abort path only

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int M = g.M, N = g.N;
    const int num_kb = g.K / BK;
    const int tiles_n = N / BN, tiles_m = (M + TM - 1) / TM;
    const int num_tiles = tiles_n * tiles_m;

    if (threadIdx.x == 0) {
        for (int s = 0; s < cfg::STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(accf0 + 8 * b, 1);
            mbar_init(acce0 + 8 * b, PAIR ? 8 : 4);  // one arrival per epilogue warp (of both CTAs)
        }
        mbar_init(drain_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0 && lane == 0) {  // descriptor fetch off the critical path
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
        if (EPI == EPI_STORE || EPI == EPI_ADD || EPI == EPI_ADDNORM)
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_c) : "memory");
        if (EPI == EPI_ADDNORM) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_hb) : "memory");
    }
    if (warp == 1) {
        if (PAIR) {  // the same warp of both CTAs allocates the same columns in both
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                             smem_u32((const void*)tmem_slot)),
                         "r"((uint32_t)cfg::TMEM_COLS)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                             smem_u32((const void*)tmem_slot)),
                         "r"((uint32_t)cfg::TMEM_COLS)
                         : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (PAIR) cluster_sync_all();  // both CTAs' barriers are initialised before either signals the other
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    // Everything above is on-chip set-up.  The weight operand W is constant for the life of the model, so the
    // producer thread fetches the W tiles of its first stages BEFORE the grid dependency resolves (they cross
    // HBM while the previous kernel drains); activations, outputs and slot tables are touched only after it.
    const bool is_producer = warp == 0 && lane == 0;
    const int num_groups = (num_kb + cfg::KG - 1) / cfg::KG;  // barrier groups per tile
    int prefetched = 0;  // groups of the first tile whose W tiles are already in flight
    if (is_producer && g.w_constant) {
        const int tile = unit;  // every CTA owns at least one tile
        const int n0 = (tile % tiles_n) * BN + (PAIR ? (int)rank * (BN / 2) : 0);
        prefetched = num_groups < cfg::GROUPS ? num_groups : cfg::GROUPS;
        for (int gi = 0; gi < prefetched; ++gi) {
            const int kb0 = gi * cfg::KG;
            const int nk = num_kb - kb0 < cfg::KG ? num_kb - kb0 : cfg::KG;
            if (!PAIR || rank == 0) mbar_expect_tx(full0 + 8 * gi, (PAIR ? 2 : 1) * nk * cfg::STAGE_BYTES);
            for (int k = 0; k < nk; ++k) {
                const uint32_t b_dst = tiles + (gi * cfg::KG + k) * cfg::STAGE_BYTES + cfg::A_BYTES;
                if (PAIR) tma_load_2d_pair(b_dst, &map_w, (kb0 + k) * BK, n0, map_to_rank(full0 + 8 * gi, 0));
                else tma_load_2d(b_dst, &map_w, (kb0 + k) * BK, n0, full0 + 8 * gi);
            }
        }
    }
    pdl_wait();

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t gc = 0;  // barrier groups issued so far
            for (int tile = unit; tile < num_tiles; tile += units) {
                const int m0 = (tile / tiles_n) * TM + (int)rank * BM;
                const int n0 = (tile % tiles_n) * BN + (PAIR ? (int)rank * (BN / 2) : 0);
                bool ok = true;
                for (int kb0 = 0; kb0 < num_kb; kb0 += cfg::KG, ++gc) {
                    const int nk = num_kb - kb0 < cfg::KG ? num_kb - kb0 : cfg::KG;
                    const uint32_t gs = gc % cfg::GROUPS, ph = (gc / cfg::GROUPS) & 1u;
                    const uint32_t bar = PAIR ? map_to_rank(full0 + 8 * gs, 0) : full0 + 8 * gs;
                    const bool first_rev = (int)gc < prefetched;
                    // first revolution of the ring: the stages are free, the barrier is armed and the W tiles
                    // are on the way; only the activation tiles are missing
                    if (!first_rev) {
                        if (!mbar_wait(empty0 + 8 * gs, ph ^ 1u, abort_flag)) {
                            raise_abort<PAIR>(abort_flag, rank);
                            atomicExch(g.error_flag, 1);
                            ok = false;
                            break;
                        }
                        // in a pair both CTAs' loads complete on the leader's barrier, which expects the bytes of both
                        if (!PAIR || rank == 0) mbar_expect_tx(full0 + 8 * gs, (PAIR ? 2 : 1) * nk * cfg::STAGE_BYTES);
                    }
                    for (int k = 0; k < nk; ++k) {
                        const uint32_t a_dst = tiles + (gs * cfg::KG + k) * cfg::STAGE_BYTES;
                        if (PAIR) {
                            tma_load_2d_pair(a_dst, &map_a, (kb0 + k) * BK, m0, bar);
                            if (!first_rev) tma_load_2d_pair(a_dst + cfg::A_BYTES, &map_w, (kb0 + k) * BK, n0, bar);
                        } else {
                            tma_load_2d(a_dst, &map_a, (kb0 + k) * BK, m0, bar);
                            if (!first_rev) tma_load_2d(a_dst + cfg::A_BYTES, &map_w, (kb0 + k) * BK, n0, bar);
                        }
                    }
                }
                if (!ok) break;
            }
            if (*abort_flag) {
                // Leaving early: the copies this thread issued must have landed before the CTA gives up its shared
                // memory.  The groups armed last are the only ones that can still be in flight; their barriers
                // complete when the bytes arrive whether or not anyone consumes them (in a pair they live in the
                // leader, which waits for both CTAs' bytes; the end-of-kernel cluster barrier holds the partner).
                if (!PAIR || rank == 0) {
                    const uint32_t first = gc > (uint32_t)cfg::GROUPS ? gc - cfg::GROUPS : 0u;
                    for (uint32_t g2 = first; g2 < gc; ++g2) {
                        const unsigned long long t0 = globaltimer_ns();
                        while (!mbar_try(full0 + 8 * (g2 % cfg::GROUPS), (g2 / cfg::GROUPS) & 1u))
                            if (globaltimer_ns() - t0 > 1000000000ull) break;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0 && rank == 0) {  // in a pair only the leader issues
            constexpr uint32_t idesc = umma_idesc(BN, TM);
            const uint64_t desc_a0 = umma_desc(tiles);  // A tile of stage 0; every other operand tile by offset
            uint32_t gc = 0, j = 0;
            for (int tile = unit; tile < num_tiles; tile += units, ++j) {
                const uint32_t buf = j & 1u, aph = (j >> 1) & 1u;
                bool ok = mbar_wait(acce0 + 8 * buf, aph ^ 1u, abort_flag);  // epilogue drained this accumulator
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tmem_d = tmem_base + buf * BN;
                for (int kb0 = 0; kb0 < num_kb && ok; kb0 += cfg::KG, ++gc) {
                    const int nk = num_kb - kb0 < cfg::KG ? num_kb - kb0 : cfg::KG;
                    const uint32_t gs = gc % cfg::GROUPS, ph = (gc / cfg::GROUPS) & 1u;
                    if (!mbar_wait(full0 + 8 * gs, ph, abort_flag)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    // descriptors by increments of the 14-bit start-address field (16-byte units; the ring lies
                    // below 256 KB, so the field never carries): + STAGE_BYTES per k-block, + 32 bytes per MMA
                    uint64_t da = desc_a0 + (uint64_t)(gs * cfg::KG * (cfg::STAGE_BYTES >> 4));
                    uint64_t db = da + (uint64_t)(cfg::A_BYTES >> 4);
                    for (int kk = 0; kk < nk; ++kk) {
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k) {
                            const uint32_t acc = (kb0 | kk | k) != 0 ? 1u : 0u;
                            if (PAIR) umma_f16_pair(tmem_d, da + 2 * k, db + 2 * k, idesc, acc);
                            else umma_f16(tmem_d, da + 2 * k, db + 2 * k, idesc, acc);
                        }
                        da += (uint64_t)(cfg::STAGE_BYTES >> 4);
                        db += (uint64_t)(cfg::STAGE_BYTES >> 4);
                    }
                    // frees the group's stages (in both CTAs of a pair) once these MMAs have read them
                    if (PAIR) umma_commit_pair(empty0 + 8 * gs);
                    else umma_commit(empty0 + 8 * gs);
                }
                if (!ok) {
                    raise_abort<PAIR>(abort_flag, rank);
                    atomicExch(g.error_flag, 2);
                    break;
                }
                if (PAIR) umma_commit_pair(accf0 + 8 * buf);  // accumulator complete
                else umma_commit(accf0 + 8 * buf);
            }
            if (*abort_flag) {
                // Leaving early: the MMAs issued so far must have completed before TMEM and the operand ring are
                // released.  A commit on a barrier of its own completes when they have.
                if (PAIR)
                    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                                     drain_bar)
                                 : "memory");
                else
                    umma_commit(drain_bar);
                const unsigned long long t0 = globaltimer_ns();
                while (!mbar_try(drain_bar, 0u))
                    if (globaltimer_ns() - t0 > 1000000000ull) break;
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps 2..5
        const int quarter = warp & 3;  // TMEM lanes 32*quarter .. 32*quarter+31 belong to this warp
        uint32_t j = 0, nchunk = 0;
        for (int tile = unit; tile < num_tiles; tile += units, ++j) {
            const int m0 = (tile / tiles_n) * TM + (int)rank * BM, n0 = (tile % tiles_n) * BN;
            const uint32_t buf = j & 1u, aph = (j >> 1) & 1u;
            const int row = m0 + quarter * 32 + lane;
            const uint32_t tbase = tmem_base + buf * BN + ((uint32_t)(quarter * 32) << 16);
            // what the tile's rows need from global memory is requested before the accumulator is waited for
            // row factor of the folded RMSNorm: the partial sums of squares of this row of A, added in a fixed order
            float rscale = 1.0f;
            if (EPI != EPI_ADD && EPI != EPI_ADDNORM && g.ssq_in != nullptr && row < M) {
                const float2* pp = reinterpret_cast<const float2*>(g.ssq_in + (size_t)row * g.ssq_n);
                float ss = 0.f;
                for (int v = 0; v < g.ssq_n / 2; ++v) {
                    const float2 t = pp[v];
                    ss += t.x;
                    ss += t.y;
                }
                rscale = 1.0f / sqrtf(ss * g.inv_dim + g.eps);
            }
            // ADDNORM: the residual values this thread's row adds to, fetched three 32-column chunks ahead through a
            // ring of four register buffers (a chunk is 128 contiguous bytes of the row; the first three are
            // requested before the accumulator is waited for)
            constexpr int UNR = EPI == EPI_ADDNORM ? 4 : 1;  // chunks per unrolled group: static ring indices
            float4 hbuf[UNR][8];
            if (EPI == EPI_ADDNORM) {
#pragma unroll
                for (int u = 0; u < 3; ++u)
#pragma unroll
                    for (int v = 0; v < 8; ++v) hbuf[u % UNR][v] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (row < M) {
#pragma unroll
                    for (int u = 0; u < 3; ++u)
                        if (u * 32 < BN) {
                            const float4* hp = reinterpret_cast<const float4*>(g.C + (size_t)row * N + n0 + u * 32);
#pragma unroll
                            for (int v = 0; v < 8; ++v) hbuf[u % UNR][v] = hp[v];
                        }
                }
            }
            if (!mbar_wait(accf0 + 8 * buf, aph, abort_flag, g.acc_wait_ns ? g.acc_wait_ns : 1000000000ull)) {
                if (lane == 0) {
                    raise_abort<PAIR>(abort_flag, rank);
                    atomicExch(g.error_flag, 3);
                }
                break;
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

            RowDst rd;
            rd.valid = row < M;
            rd.s = 0;
            rd.kvoff = 0;
            if (EPI == EPI_QKV && rd.valid) {
                const State& st = g.st;
                const int i = row % st.W;
                const int slot = (row / st.W) % g.S;
                const int br = row / (st.W * g.S);
                rd.valid = i < st.slot_n[slot];
                if (rd.valid) {
                    rd.s = st.slot_c[slot] + i;
                    rd.kvoff = g.kv.offset(g.layer, br * st.Bmax + st.slot_img[slot], rd.s);
                }
            }
            // cos/sin of this row's sequence index, fetched once per tile (all loads in flight together):
            // rotation pairs 0..15 and 16..31 of a head (head sizes 64: both halves; 32: the first)
            float4 rope_lo[8], rope_hi[8];
            if (EPI == EPI_QKV && rd.valid && n0 < 2 * g.st.D) {
                const int half = g.st.dh / 2;
                const float4* tab = reinterpret_cast<const float4*>(g.rope_cs + (size_t)rd.s * half * 2);
#pragma unroll
                for (int v = 0; v < 8; ++v) rope_lo[v] = tab[v];
                if (half > 16) {
#pragma unroll
                    for (int v = 0; v < 8; ++v) rope_hi[v] = tab[8 + v];
                }
            }
#pragma unroll 1
            for (int cg = 0; cg < BN; cg += 32 * UNR) {
              float ssq4[UNR];  // ADDNORM: sums of squares of this group's chunks
#pragma unroll
              for (int u = 0; u < UNR; ++u) ssq4[u] = 0.f;
#pragma unroll
              for (int u = 0; u < UNR; ++u) {
                const int c0 = cg + 32 * u;
                if (c0 >= BN) continue;
                uint32_t r[32];
                tmem_ld32(tbase + (uint32_t)c0, r);
                const int col = n0 + c0;
                if (EPI == EPI_ADDNORM) {
                    // this warp's staging: two buffers of (fp32 tile 4 KB, swizzled | bf16 tile 2 KB, dense)
                    const uint32_t sb32 =
                        staging + (uint32_t)(warp - 2) * (uint32_t)cfg::WARP_STAGING + (uint32_t)(nchunk++ & 1u) * 6144u;
                    const uint32_t sb16 = sb32 + 4096u;
                    float4 hcur[8];
#pragma unroll
                    for (int v = 0; v < 8; ++v) hcur[v] = hbuf[u][v];
                    // new residual = old + acc (one fp32 addition per element, as the reduce-add form did)
                    float ss = 0.f;
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const float x0 = hcur[v].x + __uint_as_float(r[4 * v]);
                        const float x1 = hcur[v].y + __uint_as_float(r[4 * v + 1]);
                        const float x2 = hcur[v].z + __uint_as_float(r[4 * v + 2]);
                        const float x3 = hcur[v].w + __uint_as_float(r[4 * v + 3]);
                        ss += x0 * x0;
                        ss += x1 * x1;
                        ss += x2 * x2;
                        ss += x3 * x3;
                        r[4 * v] = __float_as_uint(x0);
                        r[4 * v + 1] = __float_as_uint(x1);
                        r[4 * v + 2] = __float_as_uint(x2);
                        r[4 * v + 3] = __float_as_uint(x3);
                    }
                    ssq4[u] = ss;
                    // one bulk tensor store per tile (the pair is one bulk group: the buffer used two chunks ago is
                    // free once at most one group is still reading); rows past the buffers' capacity are clipped
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const uint32_t addr = sb32 + (uint32_t)lane * 128u + (uint32_t)((v ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r[4 * v]),
                                     "r"(r[4 * v + 1]), "r"(r[4 * v + 2]), "r"(r[4 * v + 3])
                                     : "memory");
                    }
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        const uint32_t p0 = pack_bf16x2(__uint_as_float(r[8 * v]), __uint_as_float(r[8 * v + 1]));
                        const uint32_t p1 = pack_bf16x2(__uint_as_float(r[8 * v + 2]), __uint_as_float(r[8 * v + 3]));
                        const uint32_t p2 = pack_bf16x2(__uint_as_float(r[8 * v + 4]), __uint_as_float(r[8 * v + 5]));
                        const uint32_t p3 = pack_bf16x2(__uint_as_float(r[8 * v + 6]), __uint_as_float(r[8 * v + 7]));
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(sb16 + (uint32_t)lane * 64u +
                                                                                    (uint32_t)v * 16u),
                                     "r"(p0), "r"(p1), "r"(p2), "r"(p3)
                                     : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0 && m0 + quarter * 32 < M) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                                         &map_c),
                                     "r"(col), "r"(m0 + quarter * 32), "r"(sb32)
                                     : "memory");
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                                         &map_hb),
                                     "r"(col), "r"(m0 + quarter * 32), "r"(sb16)
                                     : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                    // The chunk three ahead takes the register slot this chunk has freed.  Requested only now, behind
                    // the proxy fence above: a fence waits for the loads its thread has in flight, so a request in
                    // front of it would cost the fence a full memory latency per chunk.
                    if (c0 + 96 < BN && row < M) {
                        const float4* hp = reinterpret_cast<const float4*>(g.C + (size_t)row * N + col + 96);
#pragma unroll
                        for (int v = 0; v < 8; ++v) hbuf[(u + 3) % UNR][v] = hp[v];
                    }
                    continue;
                }
                if (EPI == EPI_STORE && g.ssq_in != nullptr) {
#pragma unroll
                    for (int v = 0; v < 32; ++v) r[v] = __float_as_uint(__uint_as_float(r[v]) * rscale);
                }
                if (EPI == EPI_STORE || EPI == EPI_ADD) {
                    // registers -> swizzled staging tile (32 rows x 128 bytes) -> one TMA store / reduce-add
                    // of the 32 x 32 block; rows past M are clipped by the tensor map
                    const uint32_t sbuf = staging + (uint32_t)((warp - 2) * 2 + (int)(nchunk++ & 1u)) * 4096u;
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    __syncwarp();
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const uint32_t addr = sbuf + (uint32_t)lane * 128u + (uint32_t)((v ^ (lane & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r[4 * v]),
                                     "r"(r[4 * v + 1]), "r"(r[4 * v + 2]), "r"(r[4 * v + 3])
                                     : "memory");
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0 && m0 + quarter * 32 < M) {
                        if (EPI == EPI_ADD)
                            asm volatile(
                                "cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group "
                                "[%0, {%1, %2}], [%3];" ::"l"(&map_c),
                                "r"(col), "r"(m0 + quarter * 32), "r"(sbuf)
                                : "memory");
                        else
                            asm volatile(
                                "cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                                    &map_c),
                                "r"(col), "r"(m0 + quarter * 32), "r"(sbuf)
                                : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                    continue;
                }
                if (!rd.valid) continue;
                if (EPI == EPI_SWIGLU) {
                    // columns (2f, 2f+1) = (gate_f, up_f)
                    uint4* dst = reinterpret_cast<uint4*>(g.out + (size_t)row * (N / 2) + col / 2);
                    uint32_t o[8];
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const float g0 = __uint_as_float(r[4 * v]) * rscale, u0 = __uint_as_float(r[4 * v + 1]) * rscale;
                        const float g1 = __uint_as_float(r[4 * v + 2]) * rscale, u1 = __uint_as_float(r[4 * v + 3]) * rscale;
                        // silu(g) * u with ex2.approx and rcp.approx (about 1e-6 relative, far below bf16)
                        o[v] = pack_bf16x2(__fdividef(g0, 1.0f + __expf(-g0)) * u0,
                                           __fdividef(g1, 1.0f + __expf(-g1)) * u1);
                    }
                    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
                } else {  // EPI_QKV
                    const State& st = g.st;
                    const int D = st.D;
                    const int sec = col / D, cs = col % D;  // 0 q, 1 k, 2 v; a tile never straddles sections
                    uint32_t o[16];
                    if (sec < 2) {
                        // the chunk's 16 rotation pairs: first or second half of the row's cos/sin table
                        const bool hi = ((cs % st.dh) / 2) >= 16;
#pragma unroll
                        for (int v = 0; v < 8; ++v) {
                            const float4 t = hi ? rope_hi[v] : rope_lo[v];  // cos, sin of pairs 2v and 2v+1
                            const float a0 = __uint_as_float(r[4 * v]) * rscale, b0 = __uint_as_float(r[4 * v + 1]) * rscale;
                            const float a1 = __uint_as_float(r[4 * v + 2]) * rscale, b1 = __uint_as_float(r[4 * v + 3]) * rscale;
                            o[2 * v] = pack_bf16x2(a0 * t.x - b0 * t.y, a0 * t.y + b0 * t.x);
                            o[2 * v + 1] = pack_bf16x2(a1 * t.z - b1 * t.w, a1 * t.w + b1 * t.z);
                        }
                    } else {
#pragma unroll
                        for (int v = 0; v < 16; ++v)
                            o[v] = pack_bf16x2(__uint_as_float(r[2 * v]) * rscale, __uint_as_float(r[2 * v + 1]) * rscale);
                    }
                    bf16* base = sec == 0 ? g.out + (size_t)row * D + cs
                                          : (bf16*)(sec == 1 ? g.kv.k : g.kv.v) + rd.kvoff + cs;
                    uint4* dst = reinterpret_cast<uint4*>(base);
#pragma unroll
                    for (int v = 0; v < 4; ++v) dst[v] = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
                }
              }
              if (EPI == EPI_ADDNORM && row < M) {  // the group's partial sums: 16 contiguous bytes per row
                  float* sp = g.ssq_out + (size_t)row * (N / 32) + (n0 + cg) / 32;
                  if (BN >= 128) {
                      *reinterpret_cast<float4*>(sp) = make_float4(ssq4[0], ssq4[1 % UNR], ssq4[2 % UNR], ssq4[3 % UNR]);
                  } else {
#pragma unroll
                      for (int u = 0; u < UNR; ++u)
                          if (u * 32 < BN) sp[u] = ssq4[u];
                  }
              }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                if (PAIR) mbar_arrive_cluster(map_to_rank(acce0 + 8 * buf, 0));  // the leader's MMA thread waits
                else mbar_arrive(acce0 + 8 * buf);
            }
        }
        // the staging tiles must have been read before shared memory is released; the global writes
        // themselves complete like any other store before dependent kernels pass their grid dependency
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    }
    __syncwarp();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (PAIR) cluster_sync_all();  // neither CTA leaves while the other may still read its tiles or barriers
    if (warp == 1) {
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                         "r"((uint32_t)cfg::TMEM_COLS)
                         : "memory");
        else
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

// Encoded tensor maps are cached by (address, extents, box, type): encoding costs microseconds on the host,
// and a round issues hundreds of GEMMs over the same few buffers.
struct MapKey {
    const void* base;
    int rows, inner, box_rows, kind;
    bool operator==(const MapKey& o) const {
        return base == o.base && rows == o.rows && inner == o.inner && box_rows == o.box_rows && kind == o.kind;
    }
};
struct MapKeyHash {
    size_t operator()(const MapKey& k) const {
        size_t h = std::hash<const void*>()(k.base);
        h = h * 1000003u ^ (size_t)k.rows;
        h = h * 1000003u ^ (size_t)k.inner;
        h = h * 1000003u ^ (size_t)(k.box_rows * 4 + k.kind);
        return h;
    }
};
std::mutex g_map_mu;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_map_cache;

bool cached_map(CUtensorMap* out, const MapKey& key, bool (*encode)(CUtensorMap*, const void*, int, int, int)) {
    std::lock_guard<std::mutex> lock(g_map_mu);
    auto it = g_map_cache.find(key);
    if (it != g_map_cache.end()) {
        *out = it->second;
        return true;
    }
    if (g_map_cache.size() > 4096) g_map_cache.clear();
    if (!encode(out, key.base, key.rows, key.inner, key.box_rows)) return false;
    g_map_cache.emplace(key, *out);
    return true;
}

// 2D bf16 row-major [rows, K] tensor, box = [box_rows, 64], 128-byte swizzle, zero fill out of bounds.
bool encode_map_ab(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
    EncodeFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int num_sms() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

bool make_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
    return cached_map(map, MapKey{base, rows, K, box_rows, 0}, encode_map_ab);
}

// fp32 row-major [rows, N] output, box = 32 columns (128 bytes) x 32 rows, 128-byte swizzle.
bool encode_map_c(CUtensorMap* map, const void* base, int rows, int N, int) {
    EncodeFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)N * 4};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 row-major [rows, N] output, box = 32 columns (64 bytes) x 32 rows, no swizzle (dense 2 KB tile).
bool encode_map_hb(CUtensorMap* map, const void* base, int rows, int N, int) {
    EncodeFn enc = get_encode();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)N * 2};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_map_c(CUtensorMap* map, const float* base, int rows, int N) {
    return cached_map(map, MapKey{base, rows, N, 32, 1}, encode_map_c);
}

template <int BN, int EPI>
cudaError_t launch(const CUtensorMap& ma, const CUtensorMap& mw, const CUtensorMap& mc, const CUtensorMap& mh,
                   const GemmArgs& g, cudaStream_t s) {
    static int configured[64] = {0};
    using cfg = Cfg<BN, false, EPI == EPI_ADDNORM>;
    cudaError_t e0 = ensure_dynamic_smem(k_gemm_tcgen05<BN, EPI, false>, cfg::SMEM, configured);
    if (e0 != cudaSuccess) return e0;
    const int tiles = (g.N / BN) * ((g.M + BM - 1) / BM);
    const int grid = tiles < num_sms() ? tiles : num_sms();
    return launch_k(k_gemm_tcgen05<BN, EPI, false>, dim3(grid), dim3(NUM_THREADS), (size_t)cfg::SMEM, s, ma, mw,
                    mc, mh, g);
}

// CTA pairs: 256 x BN tiles (BN = 256 or 128), one cluster of two CTAs per pair of SMs.
template <int BN, int EPI>
cudaError_t launch_pair(const CUtensorMap& ma, const CUtensorMap& mw, const CUtensorMap& mc, const CUtensorMap& mh,
                        const GemmArgs& g, cudaStream_t s) {
    static int configured[64] = {0};
    using cfg = Cfg<BN, true, EPI == EPI_ADDNORM>;
    cudaError_t e0 = ensure_dynamic_smem(k_gemm_tcgen05<BN, EPI, true>, cfg::SMEM, configured);
    if (e0 != cudaSuccess) return e0;
    const int tiles = (g.N / BN) * ((g.M + 2 * BM - 1) / (2 * BM));
    const int pairs = num_sms() / 2;
    const int grid = 2 * (tiles < pairs ? tiles : pairs);
    return launch_kc(k_gemm_tcgen05<BN, EPI, true>, dim3(grid), dim3(NUM_THREADS), (size_t)cfg::SMEM, s, 2,
                     ma, mw, mc, mh, g);
}

template <int EPI>
cudaError_t launch_bn(int bn, const CUtensorMap& ma, const CUtensorMap& mw, const CUtensorMap& mc,
                      const CUtensorMap& mh, const GemmArgs& g, cudaStream_t s) {
    switch (bn) {
        case 32: return launch<32, EPI>(ma, mw, mc, mh, g, s);
        case 64: return launch<64, EPI>(ma, mw, mc, mh, g, s);
        case 128: return launch<128, EPI>(ma, mw, mc, mh, g, s);
        case 512: return launch_pair<256, EPI>(ma, mw, mc, mh, g, s);  // 256 x 256 on a CTA pair
        case 640: return launch_pair<128, EPI>(ma, mw, mc, mh, g, s);  // 256 x 128 on a CTA pair
        default: return launch<256, EPI>(ma, mw, mc, mh, g, s);
    }
}

// m_cap >= M: row extent given to the A and C tensor maps (the capacity of the caller's buffers), so that one
// cached map serves every M; rows between M and m_cap are padding (read as they are, never stored past M's
// last 32-row block).  0: use M.
int run(int epi, const bf16* A, const bf16* W, GemmArgs& g, int force_bn, int max_bn, int m_cap, cudaStream_t s,
        char* err, size_t errlen) {
    const int M = g.M, N = g.N, K = g.K;
    if (M <= 0) return 0;
    if (K % BK != 0 || N % 32 != 0 || (((uintptr_t)A | (uintptr_t)W) & 15)) {
        snprintf(err, errlen, "gemm: needs K %% 64 == 0, N %% 32 == 0 and 16-byte aligned operands (M=%d N=%d K=%d)",
                 M, N, K);
        return -1;
    }
    if (force_bn != 0 && force_bn != 32 && force_bn != 64 && force_bn != 128 && force_bn != 256 && force_bn != 512 &&
        force_bn != 640) {
        snprintf(err, errlen, "gemm: tile %d is not one of 32, 64, 128, 256 (one CTA) or 512, 640 (CTA pair)", force_bn);
        return -1;
    }
    const bool force_pair = force_bn >= 512;
    if (force_pair) force_bn = 768 - force_bn;  // 512 -> 256 columns, 640 -> 128
    int bn = force_bn ? force_bn : gemm_tcgen05_tile_n(M, N, K);
    while (bn > max_bn) bn >>= 1;
    if (bn < 32 || N % bn != 0) {
        snprintf(err, errlen, "gemm: N=%d is not a multiple of the tile width %d", N, bn);
        return -1;
    }
    // large problems: 256 x 256 tiles on CTA pairs (a third less operand traffic per FLOP)
    // (measured on the decoder's shapes: the pair tile wins from about 0.6 tiles per CTA pair upwards)
    const long pair_tiles = N % 256 == 0 ? (long)((M + 255) / 256) * (N / 256) : 0;
    const bool pair = force_pair || (!force_bn && max_bn >= 256 && pair_tiles * 5 >= (long)(num_sms() / 2) * 3);
    if (pair && !force_pair) bn = 256;
    CUtensorMap ma, mw, mc, mh;
    memset(&mc, 0, sizeof(mc));
    memset(&mh, 0, sizeof(mh));
    const int map_rows = m_cap >= M ? m_cap : M;
    if ((epi == EPI_STORE || epi == EPI_ADD || epi == EPI_ADDNORM) && !make_map_c(&mc, g.C, map_rows, N)) {
        snprintf(err, errlen, "gemm: cuTensorMapEncodeTiled failed for the output (M=%d N=%d)", M, N);
        return -3;
    }
    if (epi == EPI_ADDNORM && !cached_map(&mh, MapKey{g.hb, map_rows, N, 32, 2}, encode_map_hb)) {
        snprintf(err, errlen, "gemm: cuTensorMapEncodeTiled failed for the bf16 output (M=%d N=%d)", M, N);
        return -3;
    }
    if (!make_map(&ma, A, map_rows, K, BM) || !make_map(&mw, W, N, K, pair ? bn / 2 : bn)) {
        snprintf(err, errlen, "gemm: cuTensorMapEncodeTiled failed (M=%d N=%d K=%d)", M, N, K);
        return -3;
    }
    cudaError_t e;
    switch (epi) {
        case EPI_STORE: e = launch_bn<EPI_STORE>(pair ? 768 - bn : bn, ma, mw, mc, mh, g, s); break;
        case EPI_ADD: e = launch_bn<EPI_ADD>(pair ? 768 - bn : bn, ma, mw, mc, mh, g, s); break;
        case EPI_SWIGLU: e = launch_bn<EPI_SWIGLU>(pair ? 768 - bn : bn, ma, mw, mc, mh, g, s); break;
        case EPI_ADDNORM: e = launch_bn<EPI_ADDNORM>(pair ? 768 - bn : bn, ma, mw, mc, mh, g, s); break;
        default: e = launch_bn<EPI_QKV>(pair ? 768 - bn : bn, ma, mw, mc, mh, g, s); break;
    }
    if (e != cudaSuccess) {
        snprintf(err, errlen, "gemm launch: %s", cudaGetErrorString(e));
        return -3;
    }
    return 0;
}

}  // namespace

// Tile width by a small cost model: waves of tiles over the SMs times the time of one tile.  Measured with the
// phase stamps of this kernel (HBSJD_GEMM_TIMELINE): a k-block costs about 0.47 us at N = 256 (MMA rate) and no
// less than about 0.19 us however narrow the tile is -- there the ring of operand stages is what limits it (the
// 16 KB activation tile of every k-block has to cross from L2 whatever N is, and about 160 KB can be in flight
// per SM); the epilogue adds about 0.15 us per 32 columns.  Large problems end up with 256 (CTA pairs), small
// ones with the widest tile that still fits one wave.
bool make_tensor_map_bf16(::CUtensorMap_st* map, const void* base, int rows, int cols, int box_rows) {
    return make_map(map, base, rows, cols, box_rows);
}

int gemm_tcgen05_tile_n(int M, int N, int K) {
    const long tiles_m = (M + BM - 1) / BM;
    const int sms = num_sms(), num_kb = K / BK;
    // enough 256-wide tiles for every SM: the wide tile has the lowest operand traffic per FLOP
    if (N % 256 == 0 && tiles_m * (N / 256) >= sms) return 256;
    int best = 0;
    float best_cost = 0.f;
    for (int bn = 256; bn >= 32; bn >>= 1) {
        if (N % bn != 0) continue;
        const long tiles = tiles_m * (N / bn);
        const long waves = (tiles + sms - 1) / sms;
        const float per_kb = fmaxf(0.19f, 0.47f * (float)bn / 256.0f);  // microseconds
        const float cost = (float)waves * (1.0f + 0.15f * (float)(bn / 32) + (float)num_kb * per_kb);
        if (best == 0 || cost < best_cost * 0.98f) {  // prefer the wider tile on a tie
            best = bn;
            best_cost = cost;
        }
    }
    return best ? best : 32;
}

int gemm_tcgen05_run(const bf16* A, const bf16* W, float* C, int M, int N, int K, int accumulate, int force_bn,
                     int m_cap, int32_t* error_flag, cudaStream_t s, char* err, size_t errlen, int w_constant,
                     unsigned int acc_wait_ns) {
    if ((uintptr_t)C & 15) {
        snprintf(err, errlen, "gemm: C must be 16-byte aligned");
        return -1;
    }
    GemmArgs g{};
    g.C = C;
    g.M = M;
    g.N = N;
    g.K = K;
    g.error_flag = error_flag;
    g.w_constant = w_constant;
    g.acc_wait_ns = acc_wait_ns;
    return run(accumulate ? EPI_ADD : EPI_STORE, A, W, g, force_bn, 256, m_cap, s, err, errlen);
}

namespace {
void set_norm(GemmArgs& g, const NormIn& nin, int K) {
    g.ssq_in = nin.ssq;
    g.ssq_n = K / 32;
    g.inv_dim = 1.0f / (float)K;
    g.eps = nin.eps;
}
}  // namespace

int gemm_tcgen05_head(const bf16* A, const bf16* W, float* C, int M, int N, int K, int m_cap, const NormIn& nin,
                      int32_t* error_flag, cudaStream_t s, char* err, size_t errlen) {
    GemmArgs g{};
    g.C = C;
    g.M = M;
    g.N = N;
    g.K = K;
    g.error_flag = error_flag;
    g.w_constant = 1;
    set_norm(g, nin, K);
    return run(EPI_STORE, A, W, g, 0, 256, m_cap, s, err, errlen);
}

int gemm_tcgen05_addnorm(const bf16* A, const bf16* W, float* h, bf16* hb, float* ssq_out, int M, int N, int K,
                         int m_cap, int32_t* error_flag, cudaStream_t s, char* err, size_t errlen) {
    if (((uintptr_t)h | (uintptr_t)hb) & 15) {
        snprintf(err, errlen, "gemm: residual buffers must be 16-byte aligned");
        return -1;
    }
    GemmArgs g{};
    g.C = h;
    g.hb = hb;
    g.ssq_out = ssq_out;
    g.M = M;
    g.N = N;
    g.K = K;
    g.error_flag = error_flag;
    g.w_constant = 1;
    return run(EPI_ADDNORM, A, W, g, 0, 256, m_cap, s, err, errlen);
}

int gemm_tcgen05_swiglu(const bf16* A, const bf16* W13_interleaved, bf16* act, int M, int F2, int K, int m_cap,
                        const NormIn& nin, int32_t* error_flag, cudaStream_t s, char* err, size_t errlen) {
    GemmArgs g{};
    set_norm(g, nin, K);
    g.out = act;
    g.M = M;
    g.N = F2;
    g.K = K;
    g.error_flag = error_flag;
    g.w_constant = 1;
    return run(EPI_SWIGLU, A, W13_interleaved, g, 0, 256, m_cap, s, err, errlen);
}

int gemm_tcgen05_qkv(const bf16* A, const bf16* Wqkv, bf16* q, const State& st, int S, int layer,
                     const float* rope_cs, const KvView& kv, int m_cap, const NormIn& nin, int32_t* error_flag,
                     cudaStream_t s, char* err, size_t errlen) {
    GemmArgs g{};
    set_norm(g, nin, st.D);
    g.out = q;
    g.M = st.nb * S * st.W;
    g.N = 3 * st.D;
    g.K = st.D;
    g.error_flag = error_flag;
    g.w_constant = 1;
    g.st = st;
    g.S = S;
    g.layer = layer;
    g.rope_cs = rope_cs;
    g.kv = kv;
    // a tile must lie inside one of the q / k / v sections and start on a rotation-pair boundary
    int max_bn = 256;
    while (st.D % max_bn != 0) max_bn >>= 1;
    return run(EPI_QKV, A, Wqkv, g, 0, max_bn, m_cap, s, err, errlen);
}

}  // namespace hbsjd
