// Ragged attention over paged per-image KV caches (Sec. 4.2 "Batched verification"), bf16, head size 64:
// persistent, warp-specialised, K/V blocks moved by TMA.
//
// Work item = one physical row (branch, slot) x HPC heads.  The items of a forward are dealt to the CTAs from a
// list sorted by context length (longest first, alternate stripes reversed), so every CTA streams about the
// same number of key blocks.  Inside a CTA
//   warp 0 (one lane)   producer: for every item, its K and V blocks of 32 keys, each one cp.async.bulk.tensor copy
//                       (128-byte swizzle) into a ring of STAGES stages, completion on mbarriers.  The producer
//                       runs ahead across item boundaries: the next item's first blocks are in flight while the
//                       current item's last ones are used.
//   warps 1..QB*HPC     consumers: warp (head, q-block) owns 16 consecutive window inputs of one head (its query
//                       fragments come straight from global memory, once per item); online
//                       softmax in fp32, products on mma.sync m16n8k16 (the work is about W FLOP per byte of K, V:
//                       far below the tensor ridge, the tensor cores only keep the math off the critical path).
// Query i of the row sits at sequence index s = c + i and attends keys 0..s: the cached prefix 0..c-1 plus the
// window's own keys c..c+i written just before by the QKV epilogue (intra-window causal mask).  Keys are
// streamed in ABSOLUTE blocks (block j = keys 32 j .. 32 j + 31), so a query's arithmetic depends on its
// sequence index only -- not on the cursor, the window or the batch: prefill chunks, Full and Compact execution
// agree bit for bit.  Rows of a block past the row's last key hold whatever the page holds (finite values of
// older rounds, zeros at first); they are masked before the softmax.
//
// Every mbarrier wait is bounded (about a second); after the limit the kernel raises the error flag, all roles
// leave their loops, the producer waits (bounded again) for its copies in flight, and the CTA returns.
// No multicast anywhere; all tensor maps cover this GPU's own memory.
#include <cuda.h>

#include <cstdio>

#include "internal.h"

namespace hbsjd {

namespace {

constexpr int DH = 64;   // head size
constexpr int KB = 32;   // keys per block
constexpr int HPC = 2;   // heads per work item
constexpr int STAGES = 3;
constexpr int TILE_BYTES = KB * DH * 2;             // one K or V tile of one head: 4 KB
constexpr int STAGE_BYTES = HPC * 2 * TILE_BYTES;   // 16 KB

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
// Bounded wait (about one second).  Returns false when it gave up or another role raised `abort`.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort) {
    if (mbar_try(bar, parity)) return true;
    unsigned long long t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (;;) {
        for (int it = 0; it < 64; ++it)
            if (mbar_try(bar, parity)) return true;
        if (*abort) return false;
        unsigned long long t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (t1 - t0 > 1000000000ull) return false;
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float c[4], const uint32_t a[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// A tile is rows of 128 bytes (64 bf16) with the 16-byte chunk index XOR-swizzled by (row & 7): the layout a TMA
// copy with 128-byte swizzle leaves in a 1024-byte aligned buffer.
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return row * 128 + ((chunk ^ (row & 7)) << 4); }

struct AttnArgs {
    State st;
    int S, layer, G;  // slots, layer, head groups (heads / HPC)
    KvView kv;
    const bf16* q;
    bf16* out;
    int32_t* error_flag;
};

// Position `pos` of the sorted item list -> work item.  Returns false for an inactive slot.
struct Item {
    int prow, crow, c, n, head0;
};
__device__ __forceinline__ bool item_at(const AttnArgs& a, const int* s_tab, int pos, Item& it) {
    const State& st = a.st;
    const int per_slot = st.nb * a.G;
    const int r = pos / per_slot, rem = pos % per_slot;
    const int br = rem / a.G, g = rem % a.G;
    const int slot = s_tab[r];  // slot with the r-th longest context
    it.n = s_tab[a.S + slot];
    if (it.n == 0) return false;
    it.c = s_tab[2 * a.S + slot];
    it.prow = br * a.S + slot;
    it.crow = br * st.Bmax + s_tab[3 * a.S + slot];
    it.head0 = g * HPC;
    return true;
}

template <int QB>
__global__ void __launch_bounds__((QB * HPC + 1) * 32, QB >= 3 ? 2 : 3) k_attention_tma(const __grid_constant__ CUtensorMap map_k,
                                                                       const __grid_constant__ CUtensorMap map_v,
                                                                       const AttnArgs a) {
    pdl_trigger();
    constexpr int NCW = QB * HPC;                 // consumer warps
    extern __shared__ unsigned char smem_raw[];
    const State& st = a.st;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;               // [STAGES][HPC][K tile | V tile]
    const uint32_t bars = ring + STAGES * STAGE_BYTES;          // full[STAGES], empty[STAGES]
    const uint32_t full0 = bars, empty0 = bars + 8 * STAGES;
    unsigned char* tail = smem_raw + (bars - raw) + 16 * STAGES;
    volatile uint32_t* abort_flag = (volatile uint32_t*)tail;
    int* s_tab = (int*)(tail + 16);  // [4][S]: order, n, c, image of every slot

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, NCW);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    }
    pdl_wait();
    for (int s = threadIdx.x; s < a.S; s += blockDim.x) {
        s_tab[s] = st.slot_order[s];
        s_tab[a.S + s] = st.slot_n[s];
        s_tab[2 * a.S + s] = st.slot_c[s];
        s_tab[3 * a.S + s] = st.slot_img[s];
    }
    __syncthreads();

    const int n_items = a.S * st.nb * a.G;
    const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
    // stripe s of the sorted list: CTA j takes position s * grid + j, in reversed order on odd stripes
    auto position = [&](int stripe) { return stripe * grid + ((stripe & 1) ? grid - 1 - cta : cta); };

    if (warp == 0) {
        // ---------------------------------------------------------------- producer
        if (lane == 0) {
            uint32_t gc = 0;  // K/V stages issued so far
            bool ok = true;
            for (int stripe = 0; ok && stripe * grid < n_items; ++stripe) {
                const int pos = position(stripe);
                Item it;
                if (pos >= n_items || !item_at(a, s_tab, pos, it)) continue;
                const int nblocks = (it.c + it.n + KB - 1) / KB;
                const int32_t* pages = a.kv.table + (size_t)it.crow * a.kv.pages_per_row;
                const int layer_row0 = a.layer * a.kv.n_pages * a.kv.page;
                for (int blk = 0; blk < nblocks; ++blk, ++gc) {
                    const uint32_t gs = gc % STAGES, ph = (gc / STAGES) & 1u;
                    if (!mbar_wait(empty0 + 8 * gs, ph ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const int key0 = blk * KB;
                    // one page holds whole blocks (the page size is a multiple of 32)
                    const int y = layer_row0 + pages[key0 / a.kv.page] * a.kv.page + key0 % a.kv.page;
                    mbar_expect_tx(full0 + 8 * gs, STAGE_BYTES);
                    for (int h = 0; h < HPC; ++h) {
                        const uint32_t dst = ring + gs * STAGE_BYTES + h * 2 * TILE_BYTES;
                        tma_load_2d(dst, &map_k, (it.head0 + h) * DH, y, full0 + 8 * gs);
                        tma_load_2d(dst + TILE_BYTES, &map_v, (it.head0 + h) * DH, y, full0 + 8 * gs);
                    }
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(a.error_flag, 5);
                // copies already issued must land before shared memory is released: wait for the stages armed last
                const uint32_t first = gc > (uint32_t)STAGES ? gc - STAGES : 0u;
                for (uint32_t g2 = first; g2 < gc; ++g2) {
                    unsigned long long t0, t1;
                    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
                    while (!mbar_try(full0 + 8 * (g2 % STAGES), (g2 / STAGES) & 1u)) {
                        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
                        if (t1 - t0 > 1000000000ull) break;
                    }
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- consumers
        const int cw = warp - 1;
        const int wh = cw / QB, wq = cw % QB;  // head within the item, q-block
        uint32_t gc = 0;
        const float sl2 = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) * log2(e)
        bool ok = true;
        for (int stripe = 0; ok && stripe * grid < n_items; ++stripe) {
            const int pos = position(stripe);
            Item it;
            if (pos >= n_items || !item_at(a, s_tab, pos, it)) continue;
            const int c = it.c, n = it.n;
            const int nblocks = (c + n + KB - 1) / KB;
            // ---- this warp's queries: 16 rows x 64 dims as A fragments.  Rows at or past n hold whatever the buffer
            // holds (finite values of older forwards): their results are never written back.
            const int i0 = wq * 16 + (lane >> 2), i1 = i0 + 8;
            uint32_t qa[4][4];
            {
                const bf16* qrow0 = a.q + ((size_t)it.prow * st.W + min(i0, st.W - 1)) * st.D + (it.head0 + wh) * DH;
                const bf16* qrow1 = a.q + ((size_t)it.prow * st.W + min(i1, st.W - 1)) * st.D + (it.head0 + wh) * DH;
#pragma unroll
                for (int kc = 0; kc < 4; ++kc) {
                    const int d = kc * 16 + (lane & 3) * 2;
                    qa[kc][0] = *reinterpret_cast<const uint32_t*>(qrow0 + d);
                    qa[kc][1] = *reinterpret_cast<const uint32_t*>(qrow1 + d);
                    qa[kc][2] = *reinterpret_cast<const uint32_t*>(qrow0 + d + 8);
                    qa[kc][3] = *reinterpret_cast<const uint32_t*>(qrow1 + d + 8);
                }
            }
            {   // the next item's query rows towards L1 while this item's keys stream (one 128-byte line per row)
                const int pos2 = (stripe + 1) * grid < n_items ? position(stripe + 1) : n_items;
                Item nx;
                if (lane < 16 && pos2 < n_items && item_at(a, s_tab, pos2, nx)) {
                    const bf16* nq = a.q + ((size_t)nx.prow * st.W + min(wq * 16 + lane, st.W - 1)) * st.D +
                                     (nx.head0 + wh) * DH;
                    asm volatile("prefetch.global.L1 [%0];" ::"l"(nq));
                }
            }
            const bool warp_active = wq * 16 < n;  // q-blocks wholly past the window only keep the ring moving
            const int s0 = c + i0, s1 = c + i1;    // sequence index of this thread's two query rows
            float o[8][4];
#pragma unroll
            for (int t = 0; t < 8; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
            float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

            for (int blk = 0; blk < nblocks; ++blk, ++gc) {
                const uint32_t gs = gc % STAGES, ph = (gc / STAGES) & 1u;
                if (!mbar_wait(full0 + 8 * gs, ph, abort_flag)) {
                    ok = false;
                    break;
                }
                const int key0 = blk * KB;
                // rows of this warp whose last visible key precedes the block contribute nothing: skip the math
                // (an all-masked block is an exact no-op of the online softmax, so skipping changes no bits)
                const int smax_warp = c + min(wq * 16 + 15, n - 1);
                if (warp_active && key0 <= smax_warp) {
                    const uint32_t kt = ring + gs * STAGE_BYTES + wh * 2 * TILE_BYTES;
                    const uint32_t vt = kt + TILE_BYTES;
                    // S = Q K^T for 32 keys: 4 n-tiles of 8 keys
                    float sc[4][4];
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt) {
                        sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
                        const int krow = nt * 8 + (lane & 7);
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            uint32_t b0, b1, b2, b3;  // k-chunks 2*half (b0,b1) and 2*half+1 (b2,b3)
                            ldmatrix_x4(kt + tile_off(krow, half * 4 + (lane >> 3)), b0, b1, b2, b3);
                            mma_bf16(sc[nt], qa[half * 2], b0, b1);
                            mma_bf16(sc[nt], qa[half * 2 + 1], b2, b3);
                        }
                    }
                    // causal mask + online softmax (rows r0 = lane/4 and r0+8; columns (lane%4)*2 + {0,1} per
                    // n-tile).  A block wholly at or before the warp's first query needs no mask; scaling a
                    // visible score is the same multiplication either way, so the two paths agree bit for bit.
                    float mx0 = m0, mx1 = m1;
                    if (key0 + KB - 1 <= c + wq * 16) {
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt) {
                            sc[nt][0] *= sl2;
                            sc[nt][1] *= sl2;
                            sc[nt][2] *= sl2;
                            sc[nt][3] *= sl2;
                            mx0 = fmaxf(mx0, fmaxf(sc[nt][0], sc[nt][1]));
                            mx1 = fmaxf(mx1, fmaxf(sc[nt][2], sc[nt][3]));
                        }
                    } else {
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt) {
                            const int key = key0 + nt * 8 + (lane & 3) * 2;
                            sc[nt][0] = key <= s0 ? sc[nt][0] * sl2 : -INFINITY;
                            sc[nt][1] = key + 1 <= s0 ? sc[nt][1] * sl2 : -INFINITY;
                            sc[nt][2] = key <= s1 ? sc[nt][2] * sl2 : -INFINITY;
                            sc[nt][3] = key + 1 <= s1 ? sc[nt][3] * sl2 : -INFINITY;
                            mx0 = fmaxf(mx0, fmaxf(sc[nt][0], sc[nt][1]));
                            mx1 = fmaxf(mx1, fmaxf(sc[nt][2], sc[nt][3]));
                        }
                    }
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                    // key 0 is visible to every query, so mx is finite from the first block on
                    const float corr0 = exp2f(m0 - mx0), corr1 = exp2f(m1 - mx1);
                    m0 = mx0;
                    m1 = mx1;
                    float rs0 = 0.f, rs1 = 0.f;
                    uint32_t pa[2][4];
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt) {
                        const float p0 = exp2f(sc[nt][0] - mx0), p1 = exp2f(sc[nt][1] - mx0);
                        const float p2 = exp2f(sc[nt][2] - mx1), p3 = exp2f(sc[nt][3] - mx1);
                        rs0 += p0 + p1;
                        rs1 += p2 + p3;
                        // the softmax weights enter the P.V product as bf16 (the normaliser keeps the fp32 values)
                        pa[nt >> 1][(nt & 1) * 2] = pack_bf16(p0, p1);
                        pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
                    }
                    rs0 += __shfl_xor_sync(0xffffffffu, rs0, 1);
                    rs0 += __shfl_xor_sync(0xffffffffu, rs0, 2);
                    rs1 += __shfl_xor_sync(0xffffffffu, rs1, 1);
                    rs1 += __shfl_xor_sync(0xffffffffu, rs1, 2);
                    l0 = l0 * corr0 + rs0;
                    l1 = l1 * corr1 + rs1;
#pragma unroll
                    for (int t = 0; t < 8; ++t) {
                        o[t][0] *= corr0;
                        o[t][1] *= corr0;
                        o[t][2] *= corr1;
                        o[t][3] *= corr1;
                    }
                    // O += P V: two k-chunks of 16 keys, 8 n-tiles of 8 dims
#pragma unroll
                    for (int kc = 0; kc < 2; ++kc) {
                        const int vrow = kc * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                        for (int dp = 0; dp < 4; ++dp) {  // pairs of n-tiles: dims dp*16 .. dp*16+15
                            uint32_t b0, b1, b2, b3;
                            ldmatrix_x4_trans(vt + tile_off(vrow, dp * 2 + (lane >> 4)), b0, b1, b2, b3);
                            mma_bf16(o[dp * 2], pa[kc], b0, b1);
                            mma_bf16(o[dp * 2 + 1], pa[kc], b2, b3);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty0 + 8 * gs);  // this warp is done with the stage
            }
            if (!ok) break;
            if (warp_active) {
                const float inv0 = 1.0f / l0, inv1 = 1.0f / l1;
                bf16* orow0 = a.out + ((size_t)it.prow * st.W + i0) * st.D + (it.head0 + wh) * DH;
                bf16* orow1 = a.out + ((size_t)it.prow * st.W + i1) * st.D + (it.head0 + wh) * DH;
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    const int d = t * 8 + (lane & 3) * 2;
                    if (i0 < n) *reinterpret_cast<uint32_t*>(orow0 + d) = pack_bf16(o[t][0] * inv0, o[t][1] * inv0);
                    if (i1 < n) *reinterpret_cast<uint32_t*>(orow1 + d) = pack_bf16(o[t][2] * inv1, o[t][3] * inv1);
                }
            }
        }
        if (!ok && lane == 0) {
            *abort_flag = 1;
            atomicExch(a.error_flag, 6);
        }
    }
    __syncthreads();  // no role leaves while another may still touch the ring or the barriers
}

template <int QB>
cudaError_t launch_qb(const CUtensorMap& mk, const CUtensorMap& mv, const AttnArgs& a, cudaStream_t s) {
    constexpr int threads = (QB * HPC + 1) * 32;
    const int smem = 1024 + STAGES * STAGE_BYTES + 16 * STAGES + 16 + 16 * a.S;
    static int configured[64] = {0};
    cudaError_t e = ensure_dynamic_smem(k_attention_tma<QB>, smem, configured);
    if (e != cudaSuccess) return e;
    // resident CTAs per SM (registers and shared memory), at most 3: the grid is exactly what is resident at once
    static int resident[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (resident[dev] == 0) {
        int n = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k_attention_tma<QB>, threads, (size_t)smem);
        if (e != cudaSuccess) return e;
        resident[dev] = n < 1 ? 1 : (n > 3 ? 3 : n);
    }
    const int per_sm = resident[dev];
    const long items = (long)a.S * a.st.nb * a.G;
    long grid = (long)device_sm_count() * per_sm;
    if (grid > items) grid = items;
    return launch_k(k_attention_tma<QB>, dim3((unsigned)grid), dim3(threads), (size_t)smem, s, mk, mv, a);
}

}  // namespace

bool attention_tma_supported(const State& st, const KvView& kv) {
    return st.dh == DH && st.W <= 64 && kv.page % KB == 0 && st.Hh % HPC == 0 && st.slot_order != nullptr;
}

int launch_attention_tma(const State& st, int S, int layer, const bf16* q, int q_rows_cap, KvView kv, bf16* out,
                         int32_t* error_flag, cudaStream_t s, char* err, size_t errlen) {
    CUtensorMap mk, mv;
    const int qb = (st.W + 15) / 16;
    const long kv_rows = (long)st.L * kv.n_pages * kv.page;
    (void)q_rows_cap;
    if (kv_rows > 0x7fffffffL || !make_tensor_map_bf16(&mk, kv.k, (int)kv_rows, st.D, KB) ||
        !make_tensor_map_bf16(&mv, kv.v, (int)kv_rows, st.D, KB)) {
        snprintf(err, errlen, "attention: cuTensorMapEncodeTiled failed");
        return -3;
    }
    AttnArgs a;
    a.st = st;
    a.S = S;
    a.layer = layer;
    a.G = st.Hh / HPC;
    a.kv = kv;
    a.out = out;
    a.q = q;
    a.error_flag = error_flag;
    cudaError_t e;
    switch (qb) {
        case 1: e = launch_qb<1>(mk, mv, a, s); break;
        case 2: e = launch_qb<2>(mk, mv, a, s); break;
        case 3: e = launch_qb<3>(mk, mv, a, s); break;
        default: e = launch_qb<4>(mk, mv, a, s); break;
    }
    if (e != cudaSuccess) {
        snprintf(err, errlen, "attention launch: %s", cudaGetErrorString(e));
        return -3;
    }
    return 0;
}

}  // namespace hbsjd
