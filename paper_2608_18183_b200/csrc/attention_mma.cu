// Ragged attention over paged per-image KV caches (Sec. 4.2 "Batched verification"), bf16, head size 64.
//
// One CTA = one physical row (branch, slot) x HPC heads; warp (head, q-block) owns 16 consecutive window
// inputs of one head.  Query i of the row sits at sequence index s = c + i and attends keys 0..s: the
// cached prefix 0..c-1 plus the window's own keys c..c+i written just before by the RoPE/KV kernel
// (intra-window causal mask).  Keys are streamed in ABSOLUTE blocks of 32 (block j = keys 32j..32j+31)
// through a cp.async ring in shared memory, so a query's arithmetic depends on its sequence index only --
// not on the cursor, the window or the batch (prefill chunks, Full and Compact execution agree bit for bit).
// The work is HBM-bound (about W FLOP per byte of K,V): tensor cores are used through mma.sync m16n8k16
// only to keep the math off the critical path; online softmax in fp32.
#include "internal.h"

namespace hbsjd {

namespace {

constexpr int DH = 64;   // head size
constexpr int KB = 32;   // keys per block
constexpr int STAGES = 3;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int sz = valid ? 16 : 0;  // src-size 0: zero fill
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
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

// Shared tile of one head and stage: K [32][64] then V [32][64] bf16, rows of 128 bytes with the 16-byte
// chunk index XOR-swizzled by (row & 7).
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return row * 128 + ((chunk ^ (row & 7)) << 4); }

template <int QB, int HPC>
__global__ void __launch_bounds__(QB * HPC * 32) k_attention_mma(State st, int S, int layer,
                                                                 const bf16* __restrict__ q, KvView kv,
                                                                 bf16* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    constexpr int NT = QB * HPC * 32;
    constexpr int HEAD_STAGE = 2 * KB * DH * 2;       // K + V bytes of one head in one stage (8 KB)
    constexpr int STAGE_BYTES = HPC * HEAD_STAGE;
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);

    const int prow = blockIdx.x;  // physical row = branch * S + slot
    const int slot = prow % S, br = prow / S;
    const int n = st.slot_n[slot];
    if (n == 0) return;
    const int c = st.slot_c[slot];
    const int img = st.slot_img[slot];
    const int crow = br * st.Bmax + img;
    const int head0 = blockIdx.y * HPC;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wh = warp / QB, wq = warp % QB;  // head within the CTA, q-block
    const int D = st.D;
    const int total_keys = c + n;
    const int nblocks = (total_keys + KB - 1) / KB;

    // ---- K/V block loader: all threads, 16-byte chunks; keys >= total_keys are zero-filled.
    // The row's page-table entries are fetched once (not once per block on the critical path of the copies),
    // and each thread's chunk coordinates are fixed for the whole kernel.
    __shared__ int s_pages[32];
    if (tid < 32 && tid < kv.pages_per_row && tid * kv.page < total_keys) s_pages[tid] = kv.table[crow * kv.pages_per_row + tid];
    __syncthreads();
    constexpr int CHUNKS = HPC * 2 * KB * 8;       // 16-byte chunks per block
    constexpr int PER_THREAD = (CHUNKS + NT - 1) / NT;  // chunks each thread copies per block
    uint32_t c_dst[PER_THREAD];                     // shared-memory offset inside a stage
    int c_src[PER_THREAD];                          // element offset from the block's first key row, K or V pool
    int c_row[PER_THREAD];
#pragma unroll
    for (int u = 0; u < PER_THREAD; ++u) {
        const int idx = tid + u * NT;
        const int chunk = idx & 7;
        const int row = (idx >> 3) & (KB - 1);
        const int kvsel = (idx >> 8) & 1;  // 0 = K, 1 = V   (8 chunks * 32 rows = 256)
        const int hh = idx >> 9;
        c_dst[u] = hh * HEAD_STAGE + kvsel * (KB * DH * 2) + tile_off(row, chunk);
        c_src[u] = row * D + (head0 + hh) * DH + chunk * 8;
        c_row[u] = idx < CHUNKS ? (row | (kvsel << 16)) : -1;
    }
    const size_t layer_base = (size_t)layer * kv.n_pages * kv.page * (size_t)D;
    auto load_block = [&](int blk, int stage) {
        const int key0 = blk * KB;
        // one page holds whole blocks (page size is a multiple of 32)
        const size_t base = layer_base + ((size_t)s_pages[key0 / kv.page] * kv.page + (key0 % kv.page)) * (size_t)D;
        const bf16* kb = (const bf16*)kv.k + base;
        const bf16* vb = (const bf16*)kv.v + base;
        const uint32_t sbase = smem_base + stage * STAGE_BYTES;
#pragma unroll
        for (int u = 0; u < PER_THREAD; ++u) {
            if (c_row[u] < 0) continue;
            const bf16* src = ((c_row[u] >> 16) ? vb : kb) + c_src[u];
            cp_async16(sbase + c_dst[u], src, key0 + (c_row[u] & 0xffff) < total_keys);
        }
    };

    // ---- this warp's queries: 16 rows x 64 dims as A fragments (rows >= n read as zero)
    const int i0 = wq * 16 + (lane >> 2), i1 = i0 + 8;
    uint32_t qa[4][4];
    {
        const bf16* qrow0 = q + ((size_t)prow * st.W + i0) * D + (head0 + wh) * DH;
        const bf16* qrow1 = q + ((size_t)prow * st.W + i1) * D + (head0 + wh) * DH;
#pragma unroll
        for (int kc = 0; kc < 4; ++kc) {
            const int d = kc * 16 + (lane & 3) * 2;
            qa[kc][0] = i0 < n ? *reinterpret_cast<const uint32_t*>(qrow0 + d) : 0u;
            qa[kc][1] = i1 < n ? *reinterpret_cast<const uint32_t*>(qrow1 + d) : 0u;
            qa[kc][2] = i0 < n ? *reinterpret_cast<const uint32_t*>(qrow0 + d + 8) : 0u;
            qa[kc][3] = i1 < n ? *reinterpret_cast<const uint32_t*>(qrow1 + d + 8) : 0u;
        }
    }
    const bool warp_active = wq * 16 < n;  // q-blocks wholly past the window only help loading
    const int s0 = c + i0, s1 = c + i1;    // sequence index of this thread's two query rows

    float o[8][4];
#pragma unroll
    for (int t = 0; t < 8; ++t) o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    const float sl2 = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) * log2(e)

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < nblocks) load_block(s, s);
        cp_async_commit();
    }

    for (int blk = 0; blk < nblocks; ++blk) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();  // block `blk` has landed for every thread; stage (blk-1)%STAGES is free again
        if (blk + STAGES - 1 < nblocks) load_block(blk + STAGES - 1, (blk + STAGES - 1) % STAGES);
        cp_async_commit();
        if (!warp_active) continue;
        const int key0 = blk * KB;
        // rows of this warp whose last visible key precedes the block contribute nothing: skip the math
        // (an all-masked block is an exact no-op of the online softmax, so skipping changes no bits)
        const int smax_warp = c + min(wq * 16 + 15, n - 1);
        if (key0 > smax_warp) continue;
        const uint32_t kt = smem_base + (blk % STAGES) * STAGE_BYTES + wh * HEAD_STAGE;
        const uint32_t vt = kt + KB * DH * 2;

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
        // causal mask + online softmax (rows r0 = lane/4 and r0+8; columns (lane%4)*2 + {0,1} per n-tile).
        // A block wholly at or before the warp's first query (key0 + 31 <= c + 16 wq) needs no mask; scaling
        // a visible score is the same multiplication either way, so the two paths agree bit for bit.
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
    cp_async_wait<0>();

    if (!warp_active) return;
    const float inv0 = 1.0f / l0, inv1 = 1.0f / l1;
    bf16* orow0 = out + ((size_t)prow * st.W + i0) * D + (head0 + wh) * DH;
    bf16* orow1 = out + ((size_t)prow * st.W + i1) * D + (head0 + wh) * DH;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const int d = t * 8 + (lane & 3) * 2;
        if (i0 < n) *reinterpret_cast<uint32_t*>(orow0 + d) = pack_bf16(o[t][0] * inv0, o[t][1] * inv0);
        if (i1 < n) *reinterpret_cast<uint32_t*>(orow1 + d) = pack_bf16(o[t][2] * inv1, o[t][3] * inv1);
    }
}

template <int QB, int HPC>
void launch_cfg(const State& st, int S, int layer, const bf16* q, KvView kv, bf16* out, cudaStream_t s) {
    constexpr int smem = STAGES * HPC * 2 * KB * DH * 2;
    static int configured[64] = {0};
    ensure_dynamic_smem(k_attention_mma<QB, HPC>, smem, configured);
    dim3 grid(st.nb * S, st.Hh / HPC);
    launch_k(k_attention_mma<QB, HPC>, dim3(grid), dim3(QB * HPC * 32), smem, s, st, S, layer, q, kv, out);
}

template <int HPC>
void launch_hpc(const State& st, int S, int layer, const bf16* q, KvView kv, bf16* out, cudaStream_t s) {
    const int qb = (st.W + 15) / 16;
    switch (qb) {
        case 1: launch_cfg<1, HPC>(st, S, layer, q, kv, out, s); break;
        case 2: launch_cfg<2, HPC>(st, S, layer, q, kv, out, s); break;
        case 3: launch_cfg<3, HPC>(st, S, layer, q, kv, out, s); break;
        default: launch_cfg<4, HPC>(st, S, layer, q, kv, out, s); break;
    }
}

}  // namespace

bool attention_mma_supported(const State& st, const KvView& kv) {
    // (the kernel keeps at most 32 page-table entries of a row in shared memory)
    return st.dh == DH && st.W <= 64 && kv.page % KB == 0 && st.Hh % 2 == 0 && kv.pages_per_row <= 32;
}

void launch_attention_mma(const State& st, int S, int layer, const bf16* q, KvView kv, bf16* out, cudaStream_t s) {
    // four heads per CTA when that still fills the machine, else two
    const long rows = (long)st.nb * S;
    static const int env_hpc = getenv("HBSJD_ATT_HPC") ? atoi(getenv("HBSJD_ATT_HPC")) : 0;  // tuning aid
    // two heads per CTA (48 KB of shared memory, four CTAs per SM) measured faster than four at every shape
    if (env_hpc == 1) return launch_hpc<1>(st, S, layer, q, kv, out, s);
    if (env_hpc == 4 && st.Hh % 4 == 0 && rows * (st.Hh / 4) >= 2 * 148) launch_hpc<4>(st, S, layer, q, kv, out, s);
    else launch_hpc<2>(st, S, layer, q, kv, out, s);
}

}  // namespace hbsjd
