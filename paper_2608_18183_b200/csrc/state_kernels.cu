// Rollout-state kernels: state init, prefill bookkeeping, initial history windows, and the fused
// probability pipeline + SJD verification (Eq. 5; greedy Eq. 4) + commit + draft refresh.
#include <cstring>
#include <mutex>

#include "../../include/hbsjd.h"
#include "accept_common.cuh"
#include "internal.h"

namespace hbsjd {

// ------------------------------------------------------------------ state init (Sec. 4.2 "Independent rollout states")
__global__ void k_init_state(State st, const int32_t* __restrict__ prefix_tokens,
                             const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ labels) {
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x;
    const int k = prefix_len[b];
    int32_t* seq = st.seq + (size_t)b * (st.T + 1);
    uint8_t* dl = st.delta + (size_t)b * (st.T + 1);
    for (int t = threadIdx.x; t <= st.T; t += blockDim.x) {
        seq[t] = (t >= 1 && t <= k) ? prefix_tokens[(size_t)b * st.T + t - 1] : 0;
        dl[t] = 0;
    }
    if (threadIdx.x == 0) {
        st.cursor[b] = k;
        st.klen[b] = k;
        st.pfill[b] = 0;
        st.qbase[b] = 0;
        st.label[b] = labels[b];
        st.m_last[b] = 0;
        st.j_last[b] = -1;
        if (b == 0)
            for (int x = 0; x < 8; ++x)
                if (x != CNT_ERROR) st.counters[x] = 0;
    }
}

void launch_init_state(const State& st, const int32_t* prefix_tokens, const int32_t* prefix_len,
                       const int32_t* labels, cudaStream_t s) {
    launch_k(k_init_state, dim3(st.B), dim3(128), 0, s, st, prefix_tokens, prefix_len, labels);
}

__global__ void k_prefill_advance(State st, int S) {
    pdl_trigger();
    pdl_wait();
    const int slot = blockIdx.x * blockDim.x + threadIdx.x;
    if (slot >= S) return;
    const int n = st.slot_n[slot];
    if (n > 0) st.pfill[st.slot_img[slot]] = st.slot_c[slot] + n;
}

void launch_prefill_advance(const State& st, int S, cudaStream_t s) {
    launch_k(k_prefill_advance, dim3((S + 127) / 128), dim3(128), 0, s, st, S);
}

// Initial window: every draft is the token H positions back, or a keyed uniform token where that
// position does not exist; all are point-mass proposals.  Reserved round value 0xFFFFFFFF.
__global__ void k_init_window(State st, uint32_t seed_lo, uint32_t seed_hi) {
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= st.B) return;
    const int c = st.cursor[b];
    if (c >= st.T) return;
    int32_t* seq = st.seq + (size_t)b * (st.T + 1);
    uint8_t* dl = st.delta + (size_t)b * (st.T + 1);
    const int n = min(st.W, st.T - c);
    for (int t = c + 1; t <= c + n - 1; ++t) {
        const int src = t - st.H;
        if (src >= 1) {
            seq[t] = seq[src];
        } else {
            uint32_t w[4];
            philox4x32_10((uint32_t)b, (uint32_t)t, 0xFFFFFFFFu, 0u, seed_lo, seed_hi, w);
            seq[t] = (int32_t)(((uint64_t)w[3] * (uint64_t)st.V) >> 32);
        }
        dl[t] = 1;
    }
}

void launch_init_window(const State& st, uint32_t seed_lo, uint32_t seed_hi, cudaStream_t s) {
    launch_k(k_init_window, dim3((st.B + 63) / 64), dim3(64), 0, s, st, seed_lo, seed_hi);
}

__global__ void k_export_tokens(State st, int32_t* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x;
    for (int t = threadIdx.x; t < st.T; t += blockDim.x)
        out[(size_t)b * st.T + t] = st.seq[(size_t)b * (st.T + 1) + t + 1];
}

void launch_export_tokens(const State& st, int32_t* out, cudaStream_t s) {
    launch_k(k_export_tokens, dim3(st.B), dim3(128), 0, s, st, out);
}

__global__ void k_calib_state(State st, int live) {
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x;
    int32_t* seq = st.seq + (size_t)b * (st.T + 1);
    uint8_t* dl = st.delta + (size_t)b * (st.T + 1);
    for (int t = threadIdx.x; t <= st.T; t += blockDim.x) {
        seq[t] = 0;
        dl[t] = 1;
    }
    if (threadIdx.x == 0) {
        st.cursor[b] = b < live ? st.T / 2 : st.T;
        st.qbase[b] = 0;
        st.label[b] = 0;
        st.klen[b] = 0;
        st.pfill[b] = 0;
    }
}

void launch_calib_state(const State& st, int live, cudaStream_t s) {
    launch_k(k_calib_state, dim3(st.B), dim3(128), 0, s, st, live);
}

// ------------------------------------------------------------------ probability pipeline + verification
// One CTA per (slot, window position i).  The guided logits of the position live in shared memory:
//   guided = l_u + s (l_c - l_u); / temperature; top-k threshold by radix select (ties kept);
//   softmax -> p_i (written out: it is the proposal q of the drafts refreshed from it);
//   accept test of draft z_{c+i+1}: u < min(1, p_i(z)/q(z))  (point-mass proposal: u < p_i(z))   [Eq. 5]
//   candidates: refreshed draft ~ p_i (word 2); replacement ~ [p_i - q]+ (word 1) if rejected, or the
//   bonus token ~ p_{n-1} (word 1) at the last position.
// Sampling is fixed-point (weights floor(a 2^30), integer running sums), so the result does not depend
// on the reduction order.  The per-image sequential part (first reject, commit, refresh) is k_commit.

constexpr int ACC_THREADS = 512;
constexpr int ACC_WARPS = ACC_THREADS / 32;

// Work area + reduction scratch behind the V floats.
struct AccShared {
    unsigned int work[SEL_BINS + SEL_CAP];  // selection histogram, then the keys of the selected bin
    float redf[ACC_WARPS];
    float red4[4][ACC_WARPS];                // min / max / sum / sum of squares per warp
    unsigned long long redu[ACC_WARPS];      // per-warp sums of the fixed-point weights of the current array
    unsigned int sel_prefix, sel_k;
    int result;
    uint32_t words[4];
    int jfirst;
};

__device__ __forceinline__ float block_max(float v, AccShared& sh) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh.redf[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = sh.redf[0];
#pragma unroll
    for (int w = 1; w < ACC_WARPS; ++w) r = fmaxf(r, sh.redf[w]);
    return r;
}

__device__ __forceinline__ float block_sum(float v, AccShared& sh) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh.redf[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
#pragma unroll
    for (int w = 0; w < ACC_WARPS; ++w) r += sh.redf[w];
    return r;
}

// Warp w owns the contiguous segment [w * seg, (w+1) * seg) of the vocabulary (seg a multiple of 128).
__device__ __forceinline__ int warp_segment(int V) { return (((V + ACC_WARPS - 1) / ACC_WARPS) + 127) / 128 * 128; }

// Fixed-point categorical pick over a[0..V) (shared memory) whose per-warp weight sums are in sh.redu
// (all threads call; ends with a barrier).  Integer running sums: the result is the smallest v whose
// inclusive sum exceeds (word * S) >> 32, whatever the order of evaluation.  -1 if the total is 0.
__device__ int block_pick(const float* a, int V, uint32_t word, AccShared& sh) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int seg = warp_segment(V);
    const int base = wid * seg;
    if (threadIdx.x == 0) sh.result = -1;
    __syncthreads();
    unsigned long long S = 0, excl = 0;
#pragma unroll
    for (int w = 0; w < ACC_WARPS; ++w) {
        if (w == wid) excl = S;
        S += sh.redu[w];
    }
    if (S != 0) {
        const unsigned long long target = ((unsigned long long)word * S) >> 32;
        if (target >= excl && target < excl + sh.redu[wid]) {  // exactly one warp
            // The warp walks its segment 1024 entries at a time: eight independent warp totals of 128
            // entries each (a lane holds four consecutive entries per step) locate the step, one scan over
            // the lanes locates the lane, and the lane resolves its four entries.
            unsigned long long run = excl;
            bool found = false;
            for (int c0 = 0; c0 < seg && !found; c0 += 1024) {
                auto lane_weight = [&](int k) -> unsigned long long {
                    const int v = base + c0 + k * 128 + lane * 4;
                    if (c0 + k * 128 >= seg || v >= V) return 0ull;
                    const float4 e = *reinterpret_cast<const float4*>(a + v);
                    return (unsigned long long)fixed_weight(e.x) + fixed_weight(e.y) + fixed_weight(e.z) +
                           fixed_weight(e.w);
                };
                unsigned long long tot[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) tot[k] = warp_sum_u64(lane_weight(k));
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    if (found) continue;
                    if (run + tot[k] > target) {
                        const unsigned long long mine = lane_weight(k);
                        unsigned long long incl = mine;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
                            if (lane >= o) incl += t;
                        }
                        const unsigned int hit = __ballot_sync(0xffffffffu, run + incl > target);
                        if (lane == __ffs(hit) - 1) {
                            const int v = base + c0 + k * 128 + lane * 4;
                            unsigned long long r = run + incl - mine;
                            int e = 0;
                            for (; e < 3; ++e) {
                                r += fixed_weight(a[v + e]);
                                if (r > target) break;
                            }
                            sh.result = v + e;
                        }
                        found = true;
                    } else {
                        run += tot[k];
                    }
                }
            }
        }
    }
    __syncthreads();
    return sh.result;
}

// Key of the k-th largest of g[0..V) by radix select, one byte per pass from the top (exact for any input).
__device__ unsigned int radix_select(const float* g, int V, unsigned int k, AccShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    unsigned int* hist = sh.work;  // [256]
    if (tid == 0) {
        sh.sel_prefix = 0u;
        sh.sel_k = k;
    }
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const unsigned int mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        for (int x = tid; x < 256; x += ACC_THREADS) hist[x] = 0u;
        __syncthreads();
        const unsigned int prefix = sh.sel_prefix;
        for (int v = tid; v < V; v += ACC_THREADS) {
            const unsigned int key = float_key(g[v]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (wid == 0) {
            // lane owns 8 consecutive bins; scan from the top bin downwards
            unsigned int cnt[8], tot = 0;
#pragma unroll
            for (int x = 0; x < 8; ++x) {
                cnt[x] = hist[lane * 8 + x];
                tot += cnt[x];
            }
            unsigned int incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int tt = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += tt;
            }
            unsigned int above = incl - tot;
            const unsigned int kk = sh.sel_k;
            if (above < kk && kk <= above + tot) {  // exactly one lane
#pragma unroll
                for (int x = 7; x >= 0; --x) {
                    if (above < kk && kk <= above + cnt[x]) {
                        sh.sel_prefix = prefix | ((unsigned int)(lane * 8 + x) << shift);
                        sh.sel_k = kk - above;
                        above = 0xFFFFFFFFu;  // done
                    } else if (above != 0xFFFFFFFFu) {
                        above += cnt[x];
                    }
                }
            }
        }
        __syncthreads();
    }
    return sh.sel_prefix;
}

// Key of the k-th largest of g[0..V), 0 < k < V, given mn = min(g), mx = max(g) and a guess `lo` of a value
// below it (any lo <= mx is safe: a wrong guess only costs a second pass).  One pass builds a 1024-bin
// histogram of the entries >= lo over [lo, mx] with a monotone binning (a higher bin holds strictly larger
// values), which locates the bin of the k-th largest and its rank inside that bin; the few entries of that
// bin are then ranked exactly against one another.  If fewer than k entries lie above lo the pass is
// repeated over [mn, mx]; a crowded bin falls back to the radix select.
__device__ unsigned int topk_threshold(const float* g, int V, unsigned int k, float mn, float mx, float lo,
                                       AccShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

    unsigned int* hist = sh.work;             // [SEL_BINS]
    unsigned int* cand = sh.work + SEL_BINS;  // [SEL_CAP] keys of the entries of the selected bin
    if (!(mx > mn)) return float_key(mn);     // all entries equal: everything is kept
    if (!(lo > mn) || !(lo < mx)) lo = mn;
    for (int attempt = 0; attempt < 2; ++attempt) {
        const float scale = (float)SEL_BINS / (mx - lo);
        for (int x = tid; x < SEL_BINS; x += ACC_THREADS) hist[x] = 0u;
        if (tid == 0) {
            sh.sel_prefix = 0xFFFFFFFFu;  // selected bin (none yet)
            sh.sel_k = 0u;                // rank of the k-th largest inside it (1-based, from the top)
            sh.result = 0;                // candidate count
        }
        __syncthreads();
        for (int v = tid * 4; v < V; v += ACC_THREADS * 4) {
            const float4 x = *reinterpret_cast<const float4*>(g + v);
            if (x.x >= lo) atomicAdd(&hist[min(SEL_BINS - 1, (int)((x.x - lo) * scale))], 1u);
            if (x.y >= lo) atomicAdd(&hist[min(SEL_BINS - 1, (int)((x.y - lo) * scale))], 1u);
            if (x.z >= lo) atomicAdd(&hist[min(SEL_BINS - 1, (int)((x.z - lo) * scale))], 1u);
            if (x.w >= lo) atomicAdd(&hist[min(SEL_BINS - 1, (int)((x.w - lo) * scale))], 1u);
        }
        __syncthreads();
        if (wid == 0) {
            unsigned int tot = 0;
            for (int x = 0; x < 32; ++x) tot += hist[lane * 32 + ((x + lane) & 31)];  // rotated: no bank conflict
            unsigned int incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int tt = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += tt;
            }
            unsigned int above = incl - tot;
            if (above < k && k <= above + tot) {  // at most one lane; none if fewer than k entries are >= lo
                for (int x = 31; x >= 0; --x) {
                    const unsigned int c = hist[lane * 32 + x];
                    if (k <= above + c) {
                        sh.sel_prefix = (unsigned int)(lane * 32 + x);
                        sh.sel_k = k - above;
                        break;
                    }
                    above += c;
                }
            }
        }
        __syncthreads();
        const unsigned int bsel = sh.sel_prefix;
        const unsigned int krem = sh.sel_k;
        if (bsel == 0xFFFFFFFFu) {  // the guess was too high: histogram the whole range
            __syncthreads();
            lo = mn;
            continue;
        }
        for (int v = tid * 4; v < V; v += ACC_THREADS * 4) {
            const float4 x4 = *reinterpret_cast<const float4*>(g + v);
            const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float x = xs[e];
                if (x >= lo && min(SEL_BINS - 1, (int)((x - lo) * scale)) == (int)bsel) {
                    const int slot = atomicAdd(&sh.result, 1);
                    if (slot < SEL_CAP) cand[slot] = float_key(x);
                }
            }
        }
        __syncthreads();
        const int nc = sh.result;
        __syncthreads();
        if (nc > SEL_CAP) return radix_select(g, V, k, sh);
        // the value with (#strictly greater) < krem <= (#greater or equal) is the krem-th largest of the bin
        for (int i = tid; i < nc; i += ACC_THREADS) {
            const unsigned int ki = cand[i];
            unsigned int gt = 0, ge = 0;
            for (int j = 0; j < nc; ++j) {
                const unsigned int kj = cand[j];
                gt += kj > ki;
                ge += kj >= ki;
            }
            if (gt < krem && krem <= ge) sh.sel_prefix = ki;  // every such thread writes the same key
        }
        __syncthreads();
        const unsigned int theta = sh.sel_prefix;
        __syncthreads();
        return theta;
    }
    return radix_select(g, V, k, sh);  // not reached: the second attempt covers every entry
}

// Block-wide min, max, sum and sum of squares (two barriers).
__device__ void block_stats(float& mn, float& mx, float& s1, float& s2, AccShared& sh) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
        s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    __syncthreads();
    if (lane == 0) {
        sh.red4[0][wid] = mn;
        sh.red4[1][wid] = mx;
        sh.red4[2][wid] = s1;
        sh.red4[3][wid] = s2;
    }
    __syncthreads();
    mn = sh.red4[0][0];
    mx = sh.red4[1][0];
    s1 = sh.red4[2][0];
    s2 = sh.red4[3][0];
#pragma unroll
    for (int w = 1; w < ACC_WARPS; ++w) {
        mn = fminf(mn, sh.red4[0][w]);
        mx = fmaxf(mx, sh.red4[1][w]);
        s1 += sh.red4[2][w];
        s2 += sh.red4[3][w];
    }
}

// Probability pipeline of one position, all threads of the CTA: guided = l_u + s (l_c - l_u); divided by
// the temperature; top-k threshold (ties kept); softmax in fp32.  Leaves p in g[0..V) (shared memory),
// writes it to pout, and leaves the per-warp fixed-point weight sums of p in sh.redu.  Ends with a barrier.
__device__ void prob_pipeline(float* g, const float* __restrict__ lc, const float* __restrict__ lu, int V,
                              float cfg_scale, float temperature, int top_k, float* __restrict__ pout,
                              AccShared& sh) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    float mn = INFINITY, mx = -INFINITY, s1 = 0.f, s2 = 0.f;
    const bool select = top_k > 0 && top_k < V;
    // The conditional logits go straight to shared memory with cp.async (every copy of the row in flight
    // at once); the unconditional ones are fetched eight float4 at a time into registers meanwhile.  A
    // thread combines exactly the elements it copied, so waiting for its own copies is enough.
    const uint32_t g_s = (uint32_t)__cvta_generic_to_shared(g);
    for (int v = tid * 4; v < V; v += ACC_THREADS * 4)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(g_s + (uint32_t)v * 4u), "l"(lc + v)
                     : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int v0 = tid * 4; v0 < V; v0 += ACC_THREADS * 4 * 8) {
        float4 y[8];
        if (lu) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int v = v0 + k * ACC_THREADS * 4;
                if (v < V) y[k] = *reinterpret_cast<const float4*>(lu + v);
            }
        }
        if (v0 == tid * 4) asm volatile("cp.async.wait_all;" ::: "memory");
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int v = v0 + k * ACC_THREADS * 4;
            if (v < V) {
                float4 x = *reinterpret_cast<float4*>(g + v);
                if (lu) {
                    x.x = __fadd_rn(y[k].x, __fmul_rn(cfg_scale, __fsub_rn(x.x, y[k].x)));
                    x.y = __fadd_rn(y[k].y, __fmul_rn(cfg_scale, __fsub_rn(x.y, y[k].y)));
                    x.z = __fadd_rn(y[k].z, __fmul_rn(cfg_scale, __fsub_rn(x.z, y[k].z)));
                    x.w = __fadd_rn(y[k].w, __fmul_rn(cfg_scale, __fsub_rn(x.w, y[k].w)));
                }
                if (temperature != 1.0f) {
                    x.x = __fdiv_rn(x.x, temperature);
                    x.y = __fdiv_rn(x.y, temperature);
                    x.z = __fdiv_rn(x.z, temperature);
                    x.w = __fdiv_rn(x.w, temperature);
                }
                *reinterpret_cast<float4*>(g + v) = x;
                mn = fminf(fminf(mn, x.x), fminf(fminf(x.y, x.z), x.w));
                mx = fmaxf(fmaxf(mx, x.x), fmaxf(fmaxf(x.y, x.z), x.w));
                if (select) {
                    s1 += (x.x + x.y) + (x.z + x.w);
                    s2 += (x.x * x.x + x.y * x.y) + (x.z * x.z + x.w * x.w);
                }
            }
        }
    }
    unsigned int theta = 0u;
    if (select) {
        block_stats(mn, mx, s1, s2, sh);  // the barriers inside also publish g
        // Guess a value below the k-th largest from a normal fit of the row: the upper-tail quantile of
        // 1.5 k / V (+ a small absolute margin), by the rational approximation of Abramowitz & Stegun
        // 26.2.23.  Only entries above the guess enter the selection histogram; the guess is verified by
        // the count and costs a second pass if it was too high.
        const float mean = s1 / (float)V;
        const float sd = sqrtf(fmaxf(s2 / (float)V - mean * mean, 0.f));
        theta = topk_threshold(g, V, (unsigned int)top_k, mn, mx, topk_guess(mean, sd, top_k, V), sh);
    } else {
        mx = block_max(mx, sh);  // the barriers inside also publish g
    }
    // exp and normalisation.  The threshold key is turned back into the float it encodes, so "kept" is one
    // float compare; ex2.approx (relative error about 1e-6 over the range used) and a multiplication by
    // 1/sum replace expf and the division: both sit well inside the probability tolerance, and every
    // downstream decision uses these very numbers.
    const float thr = theta == 0u ? -INFINITY : key_float(theta);
    float part = 0.f;
    for (int v = tid * 4; v < V; v += ACC_THREADS * 4) {
        float4 x = *reinterpret_cast<float4*>(g + v);
        x.x = x.x >= thr ? __expf(x.x - mx) : 0.f;
        x.y = x.y >= thr ? __expf(x.y - mx) : 0.f;
        x.z = x.z >= thr ? __expf(x.z - mx) : 0.f;
        x.w = x.w >= thr ? __expf(x.w - mx) : 0.f;
        *reinterpret_cast<float4*>(g + v) = x;
        part += (x.x + x.y) + (x.z + x.w);
    }
    const float den = block_sum(part, sh);
    const float inv = 1.0f / den;
    // normalise segment-wise (warp w owns [w*seg, (w+1)*seg)) so that the sampler's per-warp sums fall out
    const int seg = warp_segment(V);
    unsigned long long wsum = 0;
    for (int v = wid * seg + lane * 4; v < min(V, (wid + 1) * seg); v += 128) {
        float4 e = *reinterpret_cast<float4*>(g + v);
        e.x *= inv;
        e.y *= inv;
        e.z *= inv;
        e.w *= inv;
        *reinterpret_cast<float4*>(g + v) = e;
        *reinterpret_cast<float4*>(pout + v) = e;
        wsum += (unsigned long long)fixed_weight(e.x) + fixed_weight(e.y) + fixed_weight(e.z) + fixed_weight(e.w);
    }
    wsum = warp_sum_u64(wsum);
    if (lane == 0) sh.redu[wid] = wsum;
    __syncthreads();
}

// Stand-alone probability pipeline: one CTA per row of logits.
__global__ void __launch_bounds__(ACC_THREADS, 2) k_probs(const float* __restrict__ lc, const float* __restrict__ lu,
                                                       int V, float cfg_scale, float temperature, int top_k,
                                                       float* __restrict__ p) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* g = (float*)smem_raw;
    AccShared& sh = *(AccShared*)(smem_raw + (size_t)V * sizeof(float));
    const size_t row = blockIdx.x;
    prob_pipeline(g, lc + row * V, lu ? lu + row * V : nullptr, V, cfg_scale, temperature, top_k, p + row * V, sh);
}

__global__ void __launch_bounds__(ACC_THREADS, 2) k_prob_accept(State st, AcceptArgs a) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* g = (float*)smem_raw;  // [V]
    AccShared& sh = *(AccShared*)(smem_raw + (size_t)st.V * sizeof(float));
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int i = blockIdx.x, slot = blockIdx.y;
    const int n = st.slot_n[slot];
    if (i >= n) return;
    const int V = st.V;
    const int img = st.slot_img[slot], c = st.slot_c[slot];
    const int t = c + i + 1;  // token position this distribution decides
    const float* lc = a.logits + ((size_t)slot * st.W + i) * V;
    const float* lu = a.logits + ((size_t)(a.S + slot) * st.W + i) * V;
    if (tid == 0) philox4x32_10((uint32_t)img, (uint32_t)t, a.round, 0u, a.seed_lo, a.seed_hi, sh.words);

    float* pout = a.pcur + ((size_t)img * st.Wmax + i) * V;
    prob_pipeline(g, lc, st.nb == 2 ? lu : nullptr, V, a.cfg_scale, a.temperature, a.top_k, pout, sh);

    const size_t oidx = (size_t)img * st.Wmax + i;
    const bool last = (i == n - 1);
    int z = last ? 0 : st.seq[(size_t)img * (st.T + 1) + t];
    const bool is_delta = last ? false : (st.delta[(size_t)img * (st.T + 1) + t] != 0);
    int qi = (last || is_delta) ? 0 : (t - st.qbase[img] - 1);  // row of the previous round's probabilities
    // state that cannot be valid: record it, skip the access, treat the draft as rejected
    bool bad = false;
    if (z < 0 || z >= V) {
        if (tid == 0) atomicExch(&st.counters[CNT_ERROR], ERR_BAD_TOKEN);
        z = 0;
        bad = true;
    }
    if (qi < 0 || qi >= st.Wmax) {
        if (tid == 0) atomicExch(&st.counters[CNT_ERROR], ERR_BAD_PROPOSAL_ROW);
        qi = 0;
        bad = true;
    }
    const float* qrow = a.pprev + ((size_t)img * st.Wmax + qi) * V;

    if (a.greedy) {
        // argmax, lowest index on ties
        unsigned long long best = 0ull;
        for (int v = tid; v < V; v += ACC_THREADS) {
            const unsigned long long key =
                ((unsigned long long)__float_as_uint(g[v]) << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)v);
            best = key > best ? key : best;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        __syncthreads();
        if (lane == 0) sh.redu[wid] = best;
        __syncthreads();
        if (tid == 0) {
            unsigned long long b2 = sh.redu[0];
            for (int w = 1; w < ACC_WARPS; ++w) b2 = sh.redu[w] > b2 ? sh.redu[w] : b2;
            const int am = (int)(0xFFFFFFFFu - (unsigned)(b2 & 0xFFFFFFFFull));
            a.cand_rep[oidx] = am;
            a.cand_ref[oidx] = am;
            a.flag[oidx] = (!last && !bad && z == am) ? 1 : 0;
        }
        return;
    }

    // accept test (Eq. 5)
    if (!last) {
        if (tid == 0) {
            const float pz = g[z];
            float alpha;
            if (is_delta) alpha = pz;
            else alpha = fminf(1.0f, __fdiv_rn(pz, qrow[z]));
            const float u = (float)(sh.words[0] >> 8) * (1.0f / 16777216.0f);
            a.flag[oidx] = (!bad && u < alpha) ? 1 : 0;
        }
    }

    // refreshed draft candidate ~ p_i (weight sums already in sh.redu).  The replacement / bonus token is
    // needed at one position per image only (the first reject, else the last): k_commit draws it.
    const int ref = block_pick(g, V, sh.words[2], sh);
    if (tid == 0) a.cand_ref[oidx] = ref;
}

int accept_smem_bytes(int V) { return V * (int)sizeof(float) + (int)sizeof(AccShared); }

void launch_probs(const float* lc, const float* lu, int rows, int V, float cfg_scale, float temperature, int top_k,
                  float* p, cudaStream_t s) {
    static int configured[64] = {0};
    const int bytes = accept_smem_bytes(V);
    ensure_dynamic_smem(k_probs, bytes, configured);
    launch_k(k_probs, dim3(rows), dim3(ACC_THREADS), bytes, s, lc, lu, V, cfg_scale, temperature, top_k, p);
}

int device_sm_count() {
    static int n[64] = {0};
    int dev = 0;
    cudaGetDevice(&dev);
    dev &= 63;
    if (!n[dev]) {
        cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev);
        if (n[dev] <= 0) n[dev] = 148;
    }
    return n[dev];
}

void launch_prob_accept(const State& st, const AcceptArgs& a, cudaStream_t s) {
    if (accept_persistent_supported(st)) {
        launch_accept_persistent(st, a, device_sm_count(), s);
        return;
    }
    static int configured[64] = {0};
    const int bytes = accept_smem_bytes(st.V);
    ensure_dynamic_smem(k_prob_accept, bytes, configured);
    dim3 grid(st.W, a.S);
    launch_k(k_prob_accept, dim3(grid), dim3(ACC_THREADS), accept_smem_bytes(st.V), s, st, a);
}

// ------------------------------------------------------------------ commit + refresh (one CTA per slot)
// First reject by ballot over the accept flags.  The token committed after the accepted prefix is drawn
// here, at that one position: the replacement ~ [p_j - q]+ (point-mass proposal: p_j with the draft removed)
// at the first reject j (Eq. 5 and the sentence after it), else the bonus token ~ p_{n-1}, both with word 1
// of (image, position, round); the probabilities are read back from this round's p rows.  Thread 0 then
// commits, advances the cursor -- the KV commit is this cursor move: entries at and after the new cursor are
// recomputed by the next forward (Sec. 4.2 "Independent progress") -- and rebuilds the window.
__global__ void __launch_bounds__(ACC_THREADS) k_commit(State st, AcceptArgs a) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* g = (float*)smem_raw;  // [V]
    AccShared& sh = *(AccShared*)(smem_raw + (size_t)st.V * sizeof(float));
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int slot = blockIdx.x;
    const int n = st.slot_n[slot];
    if (n == 0) return;
    const int V = st.V;
    const int img = st.slot_img[slot], c = st.slot_c[slot];
    int32_t* seq = st.seq + (size_t)img * (st.T + 1);
    uint8_t* dl = st.delta + (size_t)img * (st.T + 1);
    if (wid == 0) {
        int j = -1;
        for (int base = 0; base < n - 1; base += 32) {
            const int i = base + lane;
            const bool rej = (i < n - 1) && (a.flag[(size_t)img * st.Wmax + i] == 0);
            const unsigned int b = __ballot_sync(0xffffffffu, rej);
            if (b) {
                j = base + __ffs(b) - 1;
                break;
            }
        }
        if (lane == 0) {
            sh.jfirst = j;
            const int t = c + (j >= 0 ? j : n - 1) + 1;
            philox4x32_10((uint32_t)img, (uint32_t)t, a.round, 0u, a.seed_lo, a.seed_hi, sh.words);
        }
    }
    __syncthreads();
    int j = sh.jfirst;
    int m = j >= 0 ? j + 1 : n;
    int tok;
    // batch-synchronous progress: an image that verified more than the batch's smallest commit keeps only that
    // many of its accepted drafts (no replacement token is drawn: the token at the new cursor was accepted)
    const bool held_back = a.m_sync != nullptr && *a.m_sync < m;
    if (held_back) {
        if (tid != 0) return;
        m = *a.m_sync;
        j = -1;
        tok = seq[c + m];
    } else if (a.greedy) {
        if (tid != 0) return;
        tok = a.cand_rep[(size_t)img * st.Wmax + (m - 1)];
    } else {
        const int is = m - 1, t = c + m;
        const float* prow = a.pcur + ((size_t)img * st.Wmax + is) * V;
        const bool reject = j >= 0;
        const int z = reject ? seq[t] : -1;
        bool is_delta = reject && dl[t] != 0;
        int qi = t - st.qbase[img] - 1;
        if (reject && !is_delta && (qi < 0 || qi >= st.Wmax)) {  // cannot be valid: record it, skip the access
            if (tid == 0) atomicExch(&st.counters[CNT_ERROR], ERR_BAD_PROPOSAL_ROW);
            is_delta = true;
        }
        const float* qrow = (reject && !is_delta) ? a.pprev + ((size_t)img * st.Wmax + qi) * V : nullptr;
        const int seg = warp_segment(V);
        const int vend = min(V, (wid + 1) * seg);
        for (int pass = 0; pass < 2; ++pass) {
            // pass 0: the residual (or p itself for the bonus token); pass 1, only after an empty residual:
            // p_j itself with the same word
            unsigned long long wsum = 0;
            for (int v0 = wid * seg + lane * 4; v0 < vend; v0 += 128 * 4) {
                float4 p4[4], q4[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int v = v0 + k * 128;
                    if (v < vend) {
                        p4[k] = *reinterpret_cast<const float4*>(prow + v);
                        if (qrow && pass == 0) q4[k] = *reinterpret_cast<const float4*>(qrow + v);
                    }
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int v = v0 + k * 128;
                    if (v < vend) {
                        float4 x = p4[k];
                        if (pass == 0) {
                            if (qrow) {
                                x.x = fmaxf(__fsub_rn(x.x, q4[k].x), 0.f);
                                x.y = fmaxf(__fsub_rn(x.y, q4[k].y), 0.f);
                                x.z = fmaxf(__fsub_rn(x.z, q4[k].z), 0.f);
                                x.w = fmaxf(__fsub_rn(x.w, q4[k].w), 0.f);
                            } else if (is_delta && (z >> 2) == (v >> 2)) {
                                if ((z & 3) == 0) x.x = 0.f;
                                if ((z & 3) == 1) x.y = 0.f;
                                if ((z & 3) == 2) x.z = 0.f;
                                if ((z & 3) == 3) x.w = 0.f;
                            }
                        }
                        *reinterpret_cast<float4*>(g + v) = x;
                        wsum += (unsigned long long)fixed_weight(x.x) + fixed_weight(x.y) + fixed_weight(x.z) +
                                fixed_weight(x.w);
                    }
                }
            }
            wsum = warp_sum_u64(wsum);
            if (lane == 0) sh.redu[wid] = wsum;
            __syncthreads();
            tok = block_pick(g, V, sh.words[1], sh);
            if (tok >= 0 || !reject) break;
        }
        if (tid != 0) return;
    }
    seq[c + m] = tok;
    dl[c + m] = 0;
    const int c2 = c + m;
    st.cursor[img] = c2;
    st.qbase[img] = c;
    st.m_last[img] = m;
    st.j_last[img] = j;
    if (c2 < st.T) {
        const int n2 = min(st.W, st.T - c2);
        for (int t = c2 + 1; t <= c2 + n2 - 1; ++t) {
            if (t <= c + n) {
                seq[t] = a.cand_ref[(size_t)img * st.Wmax + (t - c - 1)];
                dl[t] = 0;
            } else {
                const int src = t - st.H;
                if (src >= 1) {
                    seq[t] = seq[src];
                } else {
                    uint32_t w[4];
                    philox4x32_10((uint32_t)img, (uint32_t)t, a.round, 0u, a.seed_lo, a.seed_hi, w);
                    seq[t] = (int32_t)(((uint64_t)w[3] * (uint64_t)st.V) >> 32);
                }
                dl[t] = 1;
            }
        }
        atomicAdd(&st.counters[CNT_LIVE], 1);
    }
    atomicAdd(&st.counters[CNT_COMMITTED], m);
    if (j >= 0) atomicAdd(&st.counters[CNT_REJECTS], 1);
}

// One CTA: every thread walks the accept flags of its slots; block-wide minimum of the commits.
__global__ void k_sync_min(State st, AcceptArgs a, int32_t* __restrict__ m_sync) {
    pdl_trigger();
    pdl_wait();
    __shared__ int red[32];
    int best = 0x7fffffff;
    for (int slot = threadIdx.x; slot < a.S; slot += blockDim.x) {
        const int n = st.slot_n[slot];
        if (n == 0) continue;
        const int img = st.slot_img[slot];
        int m = n;
        for (int i = 0; i < n - 1; ++i)
            if (a.flag[(size_t)img * st.Wmax + i] == 0) {
                m = i + 1;
                break;
            }
        best = min(best, m);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = min(best, __shfl_xor_sync(0xffffffffu, best, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) best = min(best, red[w]);
        *m_sync = best;
    }
}

void launch_sync_min(const State& st, const AcceptArgs& a, int32_t* m_sync, cudaStream_t s) {
    launch_k(k_sync_min, dim3(1), dim3(1024), 0, s, st, a, m_sync);
}

void launch_commit(const State& st, const AcceptArgs& a, cudaStream_t s) {
    static int configured[64] = {0};
    const int bytes = accept_smem_bytes(st.V);
    ensure_dynamic_smem(k_commit, bytes, configured);
    launch_k(k_commit, dim3(a.S), dim3(ACC_THREADS), bytes, s, st, a);
}

// ------------------------------------------------------------------ stand-alone verification step
size_t verify_scratch_bytes(int batch, int window) {
    const size_t b = (size_t)batch, bw = (size_t)batch * window;
    return 4 * b * 4 + 8 * 4 + (bw + 255) / 256 * 256 + 2 * bw * 4;
}

VerifyScratch verify_scratch_carve(void* base, int batch, int window) {
    const size_t b = (size_t)batch, bw = (size_t)batch * window;
    VerifyScratch sc;
    unsigned char* p = (unsigned char*)base;
    sc.slot_img = (int32_t*)p; p += b * 4;
    sc.slot_c = (int32_t*)p;   p += b * 4;
    sc.slot_n = (int32_t*)p;   p += b * 4;
    sc.j_last = (int32_t*)p;   p += b * 4;
    sc.counters = (int32_t*)p; p += 8 * 4;
    sc.flag = p;               p += (bw + 255) / 256 * 256;
    sc.cand_rep = (int32_t*)p; p += bw * 4;
    sc.cand_ref = (int32_t*)p;
    return sc;
}

cudaError_t verify_enqueue(const VerifyDesc& d, const VerifyScratch& sc, const float* logits, const float* q_prev,
                           float* p_out, int32_t* cursor, int32_t* seq, uint8_t* delta, int32_t* qbase,
                           int32_t* m_out, cudaStream_t s) {
    State st;
    memset(&st, 0, sizeof(st));
    st.B = d.batch;
    st.T = d.T;
    st.V = d.V;
    st.Bmax = d.batch;
    st.Wmax = d.window;  // caller arrays are [batch][window][V]
    st.W = d.window;
    st.H = d.history_offset;
    st.nb = d.branches;
    st.cursor = cursor;
    st.seq = seq;
    st.delta = delta;
    st.qbase = qbase;
    st.slot_img = sc.slot_img;
    st.slot_c = sc.slot_c;
    st.slot_n = sc.slot_n;
    st.counters = sc.counters;
    st.m_last = m_out;
    st.j_last = sc.j_last;
    AcceptArgs a;
    a.logits = logits;
    a.pcur = p_out;
    a.pprev = q_prev;
    a.flag = sc.flag;
    a.cand_rep = sc.cand_rep;
    a.cand_ref = sc.cand_ref;
    a.S = d.batch;
    a.cfg_scale = d.cfg_scale;
    a.temperature = d.temperature;
    a.top_k = d.top_k;
    a.greedy = d.greedy;
    a.seed_lo = (uint32_t)(d.seed & 0xffffffffu);
    a.seed_hi = (uint32_t)(d.seed >> 32);
    a.round = d.round;
    a.m_sync = nullptr;
    // the commit counters accumulate with atomics: they must start at zero on every call
    cudaError_t e = cudaMemsetAsync(sc.counters, 0, 8 * sizeof(int32_t), s);
    if (e != cudaSuccess) return e;
    launch_setup(st, 0, 0, s);
    launch_prob_accept(st, a, s);
    launch_commit(st, a, s);
    return cudaGetLastError();
}

}  // namespace hbsjd

// ------------------------------------------------------------------ verification without any allocation
// Scratch for callers that may not allocate: a fixed device array inside the library image.  In host code
// the symbol below is only a handle; the device address is looked up once per device with
// cudaGetSymbolAddress (that device current) and handed to the kernels as an ordinary pointer.
namespace {
constexpr size_t kStaticScratchBytes = 192 * 1024;
static __device__ __align__(256) unsigned char g_verify_scratch[kStaticScratchBytes];

std::mutex g_static_mu;
void* g_static_ptr[64] = {nullptr};
}  // namespace

extern "C" int hbsjd_verify_static(void* cuda_stream, const hbsjd_verify_desc* d, const float* logits,
                                   const float* q_prev, float* p_out, int32_t* cursor, int32_t* seq, uint8_t* delta,
                                   int32_t* qbase, int32_t* m_out) {
    using namespace hbsjd;
    if (!d || !logits || !q_prev || !p_out || !cursor || !seq || !delta || !qbase || !m_out) return HBSJD_EINVAL;
    if (d->batch < 1 || d->batch > 1024 || d->window < 1 || d->window > 64 ||
        (long)d->batch * d->window > 16384 || d->T < 1 || d->V < 4 || d->V % 4 || d->V > 32768 ||
        (d->branches != 1 && d->branches != 2) || d->history_offset < 1 || !(d->temperature > 0.f) ||
        !(d->temperature < INFINITY) || !(fabsf(d->cfg_scale) < INFINITY) || d->top_k < 0)
        return HBSJD_EINVAL;
    if (verify_scratch_bytes(d->batch, d->window) > kStaticScratchBytes) return HBSJD_EINVAL;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HBSJD_ECUDA;
    void* base = nullptr;
    {
        // once per device: the array's address on the current device
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_verify_scratch) != cudaSuccess || !ptr) return HBSJD_ECUDA;
            g_static_ptr[dev] = ptr;
        }
        base = g_static_ptr[dev];
    }
    static_assert(sizeof(VerifyDesc) == sizeof(hbsjd_verify_desc), "descriptor layouts must agree");
    VerifyDesc vd;
    memcpy(&vd, d, sizeof(vd));
    const VerifyScratch sc = verify_scratch_carve(base, d->batch, d->window);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // verify_enqueue zeroes the counters; the slot tables, flags and candidates are fully rewritten for
    // every (image, position) that is read back, so stale contents of the previous call are never used
    if (verify_enqueue(vd, sc, logits, q_prev, p_out, cursor, seq, delta, qbase, m_out, s) != cudaSuccess)
        return HBSJD_ECUDA;
    // the kernels record state that cannot be valid (and skip the access): read the record back (no allocation)
    int32_t code = 0;
    if (cudaMemcpyAsync(&code, sc.counters + CNT_ERROR, sizeof(code), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return HBSJD_ECUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return HBSJD_ECUDA;
    if (code != 0) return code >= 16 ? HBSJD_EINVAL : HBSJD_ETIMEOUT;
    return HBSJD_OK;
}
