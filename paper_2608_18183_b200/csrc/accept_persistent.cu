// Probability pipeline + SJD accept test (Eq. 5; greedy Eq. 4) as a persistent kernel, for V <= 16384.
//
// One CTA of 1024 threads per SM walks the (slot, window position) items of the round.  The logits of the NEXT
// item (conditional and unconditional row, 2 x 64 KB at V = 16384) are fetched by two bulk copies into a staging
// area in shared memory, completing on an mbarrier, while the current item is processed entirely in registers:
// thread t owns the four float4 groups {c * 4096 + 4 t .. + 3}, c = 0..3, of the vocabulary from the guided
// combination to the normalised probabilities, which go to global memory straight from the registers.
//
//   guided = l_u + s (l_c - l_u); / temperature                                  (Sec. 4.2 "fused guided logits")
//   top-k threshold, ties kept: monotone 1024-bin histogram over [guess, max] of the entries above a normal-fit
//   guess of the k-th largest, bins scanned by all 32 warps, the selected bin's few entries ranked exactly
//   p = softmax in fp32; accept flag of draft z: u < min(1, p(z) / q(z)), point-mass proposal: u < p(z)   (Eq. 5)
//   refreshed-draft candidate ~ p by fixed-point sampling: integer weights floor(p 2^30), chunk totals, then an
//   ordered scan inside the one chunk that holds the target -- the result does not depend on evaluation order
//
// Five block-wide barriers per item in the usual case; warp reductions are single redux instructions on integers wherever the
// quantity is an integer or an order-preserving key.  Every reduction is a fixed tree over a fixed ownership of the vocabulary,
// so a position's probabilities are the same bits whichever CTA computes them, in Full and in Compact execution.
#include "accept_common.cuh"
#include "internal.h"

namespace hbsjd {

namespace {

constexpr int PT = 1024;          // threads per CTA
constexpr int PWARPS = PT / 32;
constexpr int NCH = 4;            // float4 groups per thread
constexpr int CHUNK = PT * 4;     // vocabulary entries per chunk
constexpr unsigned int NONE = 0xFFFFFFFFu;

struct PShared {
    unsigned int hist[SEL_BINS];
    unsigned int cand[SEL_CAP];
    unsigned int redk[2][PWARPS];  // keys of the per-warp minimum / maximum
    float fit[2];                  // sum and sum of squares of the sample the threshold guess is fitted to
    float redsum[PWARPS];
    unsigned int wtot[PWARPS];
    unsigned int csum[NCH][PWARPS];  // fixed-point weight sums per chunk and warp (a row's weights total 2^30)
    unsigned int best[2][PWARPS];    // greedy: largest probability bits, then the lowest index holding them
    unsigned int sel_bin, sel_k, ncand, theta;  // sel_bin / sel_k: state of the radix fallback
    uint32_t words[2][4];  // by item parity: a fast thread may start the next item while others finish this one
    unsigned long long mbar;
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
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

// Bounded wait (about one second).
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (;;) {
        for (int it = 0; it < 64; ++it)
            if (mbar_try_wait(bar, parity)) return true;
        unsigned long long t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (t1 - t0 > 1000000000ull) return false;
    }
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// Bin of x >= lo in the selection histogram over [lo, lo + 1024 / scale]: a monotone map (the integer nearest to
// (x - lo) * scale, read off the mantissa after adding 2^23; values beyond the range fall into the last bin).
// Monotone is all the selection needs; both passes use this same function.
__device__ __forceinline__ int sel_bin_of(float x, float lo, float scale) {
    const float f = fminf((x - lo) * scale, (float)(SEL_BINS - 1));
    return (int)(__float_as_uint(f + 8388608.0f) & 0x7FFFFFu);
}

// Key of the k-th largest of the block's register-resident values by radix select, one byte per pass from the
// top; exact for any input.  Only reached when the histogram's selected bin is too crowded for the exact ranking.
__device__ __forceinline__ unsigned int radix_select_regs(const float (&x)[NCH][4], int tid, int V, unsigned int k, PShared& sh) {
    const int lane = tid & 31, wid = tid >> 5;
    unsigned int* hist = sh.hist;  // [256] used
    __syncthreads();
    if (tid == 0) {
        sh.sel_bin = 0u;  // prefix
        sh.sel_k = k;
    }
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const unsigned int mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        const unsigned int prefix = sh.sel_bin;
#pragma unroll
        for (int c = 0; c < NCH; ++c)
            if (c * CHUNK + tid * 4 < V) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const unsigned int key = float_key(x[c][e]);
                    if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
                }
            }
        __syncthreads();
        if (wid == 0) {
            unsigned int cnt[8], tot = 0;
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                cnt[b] = hist[lane * 8 + b];
                tot += cnt[b];
            }
            unsigned int incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int tt = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += tt;
            }
            unsigned int above = incl - tot;
            const unsigned int kk = sh.sel_k;
            if (above < kk && kk <= above + tot) {
#pragma unroll
                for (int b = 7; b >= 0; --b) {
                    if (above != NONE && above < kk && kk <= above + cnt[b]) {
                        sh.sel_bin = prefix | ((unsigned int)(lane * 8 + b) << shift);
                        sh.sel_k = kk - above;
                        above = NONE;
                    } else if (above != NONE) {
                        above += cnt[b];
                    }
                }
            }
        }
        __syncthreads();
    }
    return sh.sel_bin;
}

template <bool CFG>
__global__ void __launch_bounds__(PT, 1) k_accept_persistent(State st, AcceptArgs a) {
    pdl_trigger();
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int V = st.V, W = st.W;
    float* stage_c = (float*)smem_raw;
    float* stage_u = stage_c + (CFG ? V : 0);
    PShared& sh = *(PShared*)(smem_raw + (size_t)(CFG ? 2 : 1) * V * sizeof(float));
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint32_t bar = smem_addr(&sh.mbar);
    const uint32_t row_bytes = (uint32_t)V * 4u;
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();
    __syncthreads();

    // slot tables of the round in shared memory: the item walk below reads them at every step
    int* s_n = (int*)(smem_raw + (size_t)(CFG ? 2 : 1) * V * sizeof(float) + sizeof(PShared));
    int* s_img = s_n + a.S;
    int* s_c = s_img + a.S;
    for (int sidx = tid; sidx < a.S; sidx += PT) {
        s_n[sidx] = st.slot_n[sidx];
        s_img[sidx] = st.slot_img[sidx];
        s_c[sidx] = st.slot_c[sidx];
    }
    __syncthreads();

    const int total = a.S * W;
    auto valid = [&](int it) { return (it % W) < s_n[it / W]; };
    auto issue = [&](int it) {  // thread 0: both rows of item `it` into the staging area
        const int slot = it / W, i = it % W;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar),
                     "r"(CFG ? 2u * row_bytes : row_bytes)
                     : "memory");
        bulk_load(smem_addr(stage_c), a.logits + ((size_t)slot * W + i) * V, row_bytes, bar);
        if (CFG) bulk_load(smem_addr(stage_u), a.logits + ((size_t)(a.S + slot) * W + i) * V, row_bytes, bar);
    };
    // The state an item needs besides its logits -- the draft token under test, whether its proposal is a point
    // mass, the proposal row and the proposal's entry q(z) -- sits behind three levels of dependent global loads.
    // They are issued one item ahead (token, flag and row base while the previous item starts; q(z) by the thread
    // that owns vocabulary entry z once those have landed), so that no item waits for them.
    struct Raw { int z, dl, qb; };
    auto fetch_raw = [&](int it) {
        Raw r = {0, 0, 0};
        const int slot = it / W, i = it % W;
        if (i < s_n[slot] - 1) {  // the last input of a window has no draft to verify
            const int img = s_img[slot];
            const size_t at = (size_t)img * (st.T + 1) + s_c[slot] + i + 1;
            r.z = st.seq[at];
            r.dl = st.delta[at];
            r.qb = st.qbase[img];
        }
        return r;
    };
    // q(z) of item `it` for the owning thread (1 elsewhere); records state that cannot be valid
    auto fetch_qz = [&](int it, const Raw& r) {
        const int slot = it / W, i = it % W;
        float qz = 1.0f;
        if (i < s_n[slot] - 1 && r.z >= 0 && r.z < V && ((r.z % CHUNK) >> 2) == tid && r.dl == 0 && !a.greedy) {
            const int qi = s_c[slot] + i + 1 - r.qb - 1;  // row of the previous round's probabilities
            if (qi < 0 || qi >= st.Wmax) {
                atomicExch(&st.counters[CNT_ERROR], ERR_BAD_PROPOSAL_ROW);
                qz = INFINITY;  // alpha = 0: rejected
            } else {
                qz = a.pprev[((size_t)s_img[slot] * st.Wmax + qi) * V + r.z];
            }
        }
        return qz;
    };
    int it = blockIdx.x;
    while (it < total && !valid(it)) it += gridDim.x;
    if (it < total && tid == 0) issue(it);
    uint32_t phase = 0;
    const bool select = a.top_k > 0 && a.top_k < V;
    Raw raw = {0, 0, 0};
    float qz = 1.0f;
    if (it < total) {
        raw = fetch_raw(it);
        qz = fetch_qz(it, raw);
    }
    // random words of an item (Philox keyed by image, position, round): computed one item ahead by one thread
    auto make_words = [&](int it, uint32_t* dst) {
        const int slot = it / W, i = it % W;
        philox4x32_10((uint32_t)s_img[slot], (uint32_t)(s_c[slot] + i + 1), a.round, 0u, a.seed_lo, a.seed_hi, dst);
    };
    uint32_t par = 0;  // item parity
    if (it < total && tid == PT - 32) make_words(it, sh.words[0]);
    sh.hist[tid] = 0u;  // SEL_BINS == PT
    // threshold guess carried from the previous item of this CTA: lower end and bin scale of the selection histogram
    float g_lo = 0.f, g_scale = 0.f;
    bool have_guess = false;
    __syncthreads();

    while (it < total) {
        int nxt = it + gridDim.x;
        while (nxt < total && !valid(nxt)) nxt += gridDim.x;
        Raw raw_next = {0, 0, 0};
        if (nxt < total) raw_next = fetch_raw(nxt);  // consumed after barrier (1)
        const int slot = it / W, i = it % W;
        const int n = s_n[slot], img = s_img[slot], c = s_c[slot];
        const int t = c + i + 1;  // token position this distribution decides
        const bool last = (i == n - 1);
        const size_t oidx = (size_t)img * st.Wmax + i;
        float* pout = a.pcur + oidx * V;

        int z = -1;
        bool is_delta = false, own_z = false;
        if (!last) {
            z = raw.z;
            is_delta = raw.dl != 0;
            if (z < 0 || z >= V) {
                if (tid == 0) atomicExch(&st.counters[CNT_ERROR], ERR_BAD_TOKEN);
                z = -1;
            } else {
                own_z = ((z % CHUNK) >> 2) == tid;
            }
        }
        const uint32_t* words = sh.words[par];  // written one item ahead (below), published by the barriers between
        if (tid == 0) sh.ncand = 0u;

        // ---- the item's logits have landed (bounded wait; the threads agree on its outcome at barrier (1))
        const bool ok = mbar_wait_bounded(bar, phase);
        phase ^= 1u;

        // ---- pass 1: guided logits into registers, row statistics
        float x[NCH][4];
        float mn = INFINITY, mx = -INFINITY, s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            const int v = ch * CHUNK + tid * 4;
            if (v < V) {
                float4 lc = *reinterpret_cast<const float4*>(stage_c + v);
                if (CFG) {
                    const float4 lu = *reinterpret_cast<const float4*>(stage_u + v);
                    lc.x = __fadd_rn(lu.x, __fmul_rn(a.cfg_scale, __fsub_rn(lc.x, lu.x)));
                    lc.y = __fadd_rn(lu.y, __fmul_rn(a.cfg_scale, __fsub_rn(lc.y, lu.y)));
                    lc.z = __fadd_rn(lu.z, __fmul_rn(a.cfg_scale, __fsub_rn(lc.z, lu.z)));
                    lc.w = __fadd_rn(lu.w, __fmul_rn(a.cfg_scale, __fsub_rn(lc.w, lu.w)));
                }
                if (a.temperature != 1.0f) {
                    lc.x = __fdiv_rn(lc.x, a.temperature);
                    lc.y = __fdiv_rn(lc.y, a.temperature);
                    lc.z = __fdiv_rn(lc.z, a.temperature);
                    lc.w = __fdiv_rn(lc.w, a.temperature);
                }
                x[ch][0] = lc.x; x[ch][1] = lc.y; x[ch][2] = lc.z; x[ch][3] = lc.w;
                mn = fminf(fminf(mn, lc.x), fminf(fminf(lc.y, lc.z), lc.w));
                mx = fmaxf(fmaxf(mx, lc.x), fmaxf(fmaxf(lc.y, lc.z), lc.w));
                if (select && wid == 0) {
                    s1 += (lc.x + lc.y) + (lc.z + lc.w);
                    s2 += (lc.x * lc.x + lc.y * lc.y) + (lc.z * lc.z + lc.w * lc.w);
                }
                if (have_guess) {  // selection histogram with the carried guess, verified after the barrier
                    int b4[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) b4[e] = sel_bin_of(fmaxf(x[ch][e], g_lo), g_lo, g_scale);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (x[ch][e] >= g_lo) atomicAdd(&sh.hist[b4[e]], 1u);
                }
            } else {
                x[ch][0] = x[ch][1] = x[ch][2] = x[ch][3] = -INFINITY;
            }
        }
        // minimum / maximum of the row: one warp reduction instruction each on the order-preserving keys
        {
            const unsigned int kmn = __reduce_min_sync(0xffffffffu, float_key(mn));
            const unsigned int kmx = __reduce_max_sync(0xffffffffu, float_key(mx));
            if (lane == 0) {
                sh.redk[0][wid] = kmn;
                sh.redk[1][wid] = kmx;
            }
        }
        // The threshold guess is fitted to a sample: the 128 float4 groups of warp 0 (every 32nd group of the first
        // eighth of each chunk; vocabulary order carries no structure).  Only the cost of the selection depends on it.
        int fit_n = 0;
        if (select) {
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) fit_n += max(0, min(128, V - ch * CHUNK));
            if (wid == 0) {
                s1 = warp_sum(s1);
                s2 = warp_sum(s2);
                if (lane == 0) {
                    sh.fit[0] = s1;
                    sh.fit[1] = s2;
                }
            }
        }
        // (1) staging read by everyone; partial statistics, histogram zeros and words published
        if (!__syncthreads_and(ok ? 1 : 0)) {
            if (tid == 0) atomicExch(&st.counters[CNT_ERROR], 4);
            break;  // a copy never arrived; nothing else is in flight (the next item's copies are issued below)
        }
        if (tid == 0 && nxt < total) issue(nxt);  // the next item's rows stream in behind the rest of this one
        if (tid == PT - 32 && nxt < total) make_words(nxt, sh.words[par ^ 1u]);
        float qz_next = 1.0f;
        if (nxt < total) qz_next = fetch_qz(nxt, raw_next);
        mn = key_float(__reduce_min_sync(0xffffffffu, sh.redk[0][lane]));
        mx = key_float(__reduce_max_sync(0xffffffffu, sh.redk[1][lane]));

        // ---- exact top-k threshold (ties kept).  The selection histogram covers [lo, lo + 1024 / scale] with (lo,
        // scale) from, in turn: the guess carried from this CTA's previous item (the histogram was then filled during
        // pass 1), a normal fit of this row's sample, the row's whole range.  A source whose lower end lies above
        // the k-th largest is detected by the count and the next one is tried; the result is exact whatever the source.
        float thr = -INFINITY;
        if (select) {
            if (!(mx > mn)) {
                thr = mn;  // all entries equal: everything is kept
                if (have_guess) {
                    __syncthreads();
                    sh.hist[tid] = 0u;
                }
                have_guess = false;
            } else {
                const unsigned int k = (unsigned int)a.top_k;
                unsigned int theta = 0u;
                float lo = g_lo, scale = g_scale;
                for (int source = have_guess ? 0 : 1; source < 3; ++source) {
                    if (source > 0) {
                        if (source == 1) {
                            const float mean = sh.fit[0] / (float)fit_n;
                            const float sd = sqrtf(fmaxf(sh.fit[1] / (float)fit_n - mean * mean, 0.f));
                            lo = topk_guess(mean, sd, a.top_k, V);
                            if (!(lo > mn) || !(lo < mx)) {
                                lo = mn;
                                source = 2;
                            }
                        } else {
                            lo = mn;
                        }
                        scale = (float)SEL_BINS / (mx - lo);
#pragma unroll
                        for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (x[ch][e] >= lo) atomicAdd(&sh.hist[sel_bin_of(x[ch][e], lo, scale)], 1u);
                        __syncthreads();  // (2) only without a carried guess
                    }
                    // bins from the top: warp w, lane l looks at bin 1023 - (32 w + l)
                    const unsigned int cnt = sh.hist[SEL_BINS - 1 - (wid * 32 + lane)];
                    unsigned int incl = cnt;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned int tt = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += tt;
                    }
                    if (lane == 31) sh.wtot[wid] = incl;
                    __syncthreads();  // (3)
                    // every warp locates the bin of the k-th largest by itself: first the warp-sized group of bins ...
                    unsigned int winc = sh.wtot[lane];
                    const unsigned int wcnt = winc;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned int tt = __shfl_up_sync(0xffffffffu, winc, o);
                        if (lane >= o) winc += tt;
                    }
                    const unsigned int wmask = __ballot_sync(0xffffffffu, winc >= k);
                    if (wmask == 0u) {  // fewer than k entries at or above lo: the next source (uniform decision)
                        __syncthreads();
                        sh.hist[tid] = 0u;
                        __syncthreads();
                        continue;
                    }
                    const int wsel = __ffs(wmask) - 1;
                    const unsigned int above_w = __shfl_sync(0xffffffffu, winc - wcnt, wsel);
                    // ... then the bin inside that group
                    const unsigned int bcnt = sh.hist[SEL_BINS - 1 - (wsel * 32 + lane)];
                    unsigned int binc = bcnt;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const unsigned int tt = __shfl_up_sync(0xffffffffu, binc, o);
                        if (lane >= o) binc += tt;
                    }
                    const int lsel = __ffs(__ballot_sync(0xffffffffu, above_w + binc >= k)) - 1;
                    const int bsel = SEL_BINS - 1 - (wsel * 32 + lsel);
                    const unsigned int krem = k - (above_w + __shfl_sync(0xffffffffu, binc - bcnt, lsel));
                    // entries of the selected bin: a two-compare interval test a little wider than the bin, the
                    // exact bin function only inside it (the last bin also takes everything above the range)
                    const float inv_scale = 1.0f / scale;
                    const float c_lo = fmaxf(lo, lo + ((float)bsel - 1.0f) * inv_scale);
                    const float c_hi = bsel == SEL_BINS - 1 ? INFINITY : lo + ((float)bsel + 1.0f) * inv_scale;
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (x[ch][e] >= c_lo && x[ch][e] <= c_hi && sel_bin_of(x[ch][e], lo, scale) == bsel) {
                                const unsigned int sidx = atomicAdd(&sh.ncand, 1u);
                                if (sidx < (unsigned int)SEL_CAP) sh.cand[sidx] = float_key(x[ch][e]);
                            }
                    __syncthreads();  // (5)
                    sh.hist[tid] = 0u;  // every read of the histogram is behind us: clean for the next item's pass 1
                    const int nc = (int)sh.ncand;
                    // the key with (#strictly greater) < krem <= (#greater or equal) is the krem-th largest of the bin
                    if (nc <= 32) {  // the usual case: every warp ranks the few candidates by itself
                        const unsigned int ku = lane < nc ? sh.cand[lane] : 0u;
                        unsigned int gt = 0, ge = 0;
                        for (int w2 = 0; w2 < nc; ++w2) {
                            const unsigned int kw = sh.cand[w2];
                            gt += kw > ku;
                            ge += kw >= ku;
                        }
                        const unsigned int hit = __ballot_sync(0xffffffffu, lane < nc && gt < krem && krem <= ge);
                        theta = __shfl_sync(0xffffffffu, ku, __ffs(hit) - 1);
                    } else if (nc > SEL_CAP) {
                        theta = radix_select_regs(x, tid, V, k, sh);
                        __syncthreads();
                        sh.hist[tid] = 0u;  // the radix passes used the first 256 bins
                    } else {
                        for (int u = tid; u < nc; u += PT) {
                            const unsigned int ku = sh.cand[u];
                            unsigned int gt = 0, ge = 0;
                            for (int w2 = 0; w2 < nc; ++w2) {
                                const unsigned int kw = sh.cand[w2];
                                gt += kw > ku;
                                ge += kw >= ku;
                            }
                            if (gt < krem && krem <= ge) sh.theta = ku;  // every such thread writes the same key
                        }
                        __syncthreads();  // (6)
                        theta = sh.theta;
                    }
                    break;
                }
                thr = key_float(theta);
                // the next item's guess: a lower end a little below this threshold, a top a little above this maximum
                g_lo = thr - 0.3f * (mx - thr);
                g_scale = (float)SEL_BINS / (1.4f * (mx - thr));
                have_guess = mx > thr;
            }
        }

        // ---- exp and normalisation (ex2.approx and a multiplication by 1/sum: inside the probability tolerance,
        // and every downstream decision uses these very numbers)
        float part = 0.f;
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                x[ch][e] = x[ch][e] >= thr ? __expf(x[ch][e] - mx) : 0.f;  // entries past V are -inf: 0
                part += x[ch][e];
            }
        part = warp_sum(part);
        if (lane == 0) sh.redsum[wid] = part;
        __syncthreads();  // (7)
        const float den = warp_sum(sh.redsum[lane]);
        const float inv = 1.0f / den;
        // fixed-point weights floor(p 2^30): the whole row totals 2^30 (1 + 1e-3) at most, so 32-bit sums are exact
        unsigned int wc[NCH];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            const int v = ch * CHUNK + tid * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) x[ch][e] *= inv;
            wc[ch] = fixed_weight(x[ch][0]) + fixed_weight(x[ch][1]) + fixed_weight(x[ch][2]) + fixed_weight(x[ch][3]);
            if (v < V) *reinterpret_cast<float4*>(pout + v) = make_float4(x[ch][0], x[ch][1], x[ch][2], x[ch][3]);
        }

        if (a.greedy) {
            // argmax, lowest index on ties: the largest probability bits, then the lowest index that holds them
            unsigned int bb = 0u;
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                for (int e = 0; e < 4; ++e) bb = max(bb, __float_as_uint(x[ch][e]));  // p >= 0: bits are ordered
            bb = __reduce_max_sync(0xffffffffu, bb);
            if (lane == 0) sh.best[0][wid] = bb;
            __syncthreads();  // (8)
            bb = __reduce_max_sync(0xffffffffu, sh.best[0][lane]);
            unsigned int bi = NONE;
#pragma unroll
            for (int ch = NCH - 1; ch >= 0; --ch)
#pragma unroll
                for (int e = 3; e >= 0; --e) {
                    const int v = ch * CHUNK + tid * 4 + e;
                    if (v < V && __float_as_uint(x[ch][e]) == bb) bi = (unsigned int)v;
                }
            bi = __reduce_min_sync(0xffffffffu, bi);
            if (lane == 0) sh.best[1][wid] = bi;
            __syncthreads();  // (9)
            bi = __reduce_min_sync(0xffffffffu, sh.best[1][lane]);
            if (tid == 0) {
                const int am = (int)bi;
                a.cand_rep[oidx] = am;
                a.cand_ref[oidx] = am;
                a.flag[oidx] = (!last && z == am) ? 1 : 0;
            }
        } else {
            // accept test (Eq. 5) by the owner of entry z
            if (!last && z < 0 && tid == 0) a.flag[oidx] = 0;  // invalid draft token: rejected
            if (own_z) {
                // p(z) out of the registers by a masked sum (a computed index would move the row to local memory)
                const int zc = z / CHUNK, ze = z & 3;
                float pz = 0.f;
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
                    for (int e = 0; e < 4; ++e) pz = __fmaf_rn((ch == zc && e == ze) ? 1.0f : 0.0f, x[ch][e], pz);
                const float alpha = is_delta ? pz : fminf(1.0f, __fdiv_rn(pz, qz));
                const float u = (float)(words[0] >> 8) * (1.0f / 16777216.0f);
                a.flag[oidx] = (u < alpha) ? 1 : 0;
            }
            // refreshed draft candidate ~ p (word 2): chunk totals, then the ordered scan inside one chunk
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                const unsigned int ws = __reduce_add_sync(0xffffffffu, wc[ch]);
                if (lane == 0) sh.csum[ch][wid] = ws;
            }
            __syncthreads();  // (8)
            unsigned int ctot[NCH], S = 0;
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                ctot[ch] = __reduce_add_sync(0xffffffffu, sh.csum[ch][lane]);
                S += ctot[ch];
            }
            if (S == 0) {
                if (tid == 0) a.cand_ref[oidx] = -1;
            } else {
                const unsigned int target = (unsigned int)(((unsigned long long)words[2] * S) >> 32);  // < S
                unsigned int run = 0, mine = 0, wsel = 0;
                int cs = 0;
                {
                    unsigned int start = 0;
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch) {  // the chunk whose span of the running sum holds the target
                        if (target >= start && target - start < ctot[ch]) {
                            cs = ch;
                            run = start;
                            mine = wc[ch];
                            wsel = lane < wid ? sh.csum[ch][lane] : 0u;
                        }
                        start += ctot[ch];
                    }
                }
                // position of this thread's group inside the chunk: warps before it, then lanes before it
                const unsigned int wbase = __reduce_add_sync(0xffffffffu, wsel);
                unsigned int incl = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned int tt = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += tt;
                }
                const unsigned int start = run + wbase + incl - mine;
                if (target >= start && target - start < mine) {  // exactly one thread
                    unsigned int r = start;
                    int pick = 3;
                    bool found = false;
#pragma unroll
                    for (int ch = 0; ch < NCH; ++ch)
                        if (ch == cs) {
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                r += fixed_weight(x[ch][e]);
                                if (!found && r > target) {
                                    pick = e;
                                    found = true;
                                }
                            }
                        }
                    a.cand_ref[oidx] = cs * CHUNK + tid * 4 + pick;
                }
            }
        }
        it = nxt;
        par ^= 1u;
        raw = raw_next;
        qz = qz_next;
    }
}

}  // namespace

bool accept_persistent_supported(const State& st) { return st.V <= NCH * CHUNK && st.V % 4 == 0; }

void launch_accept_persistent(const State& st, const AcceptArgs& a, int n_sms, cudaStream_t s) {
    const int nb = st.nb;
    const int bytes = nb * st.V * (int)sizeof(float) + (int)sizeof(PShared) + 3 * a.S * (int)sizeof(int);
    const int items = a.S * st.W;
    const int grid = items < n_sms ? items : n_sms;
    static int configured[2][64] = {{0}, {0}};
    if (nb == 2) {
        ensure_dynamic_smem(k_accept_persistent<true>, bytes, configured[1]);
        launch_k(k_accept_persistent<true>, dim3(grid), dim3(PT), bytes, s, st, a);
    } else {
        ensure_dynamic_smem(k_accept_persistent<false>, bytes, configured[0]);
        launch_k(k_accept_persistent<false>, dim3(grid), dim3(PT), bytes, s, st, a);
    }
}

}  // namespace hbsjd
