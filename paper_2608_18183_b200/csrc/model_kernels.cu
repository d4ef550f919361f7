// Row-wise kernels of the verifier forward (Sec. 4.2 "Batched verification"): slot set-up / compaction,
// embedding gather, RMSNorm, 2D RoPE + paged KV write, reference attention, SwiGLU, CUDA-core GEMM.
#include "internal.h"

namespace hbsjd {

// ------------------------------------------------------------------ set-up / compaction (Sec. 4.3)
// One block.  Builds the slot tables of the next forward.  Full: slot b = image b, n = 0 for inactive
// images.  Compact: active images gathered in increasing image order (block-wide exclusive scan).
__global__ void k_setup(State st, int phase, int compact) {
    pdl_trigger();
    pdl_wait();
    __shared__ int warp_tot[32];
    __shared__ int carry, sum_keys, sum_n;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid == 0) carry = sum_keys = sum_n = 0;
    __syncthreads();
    for (int base = 0; base < st.B; base += blockDim.x) {
        const int b = base + tid;
        int c = 0, n = 0;
        if (b < st.B) {
            if (phase == 0) {
                c = st.cursor[b];
                if (c < 0 || c > st.T) {  // cannot be valid: record it and leave the image out of the round
                    atomicExch(&st.counters[CNT_ERROR], 16);
                    c = st.T;
                }
                n = c < st.T ? min(st.W, st.T - c) : 0;
            } else {
                c = st.pfill[b];
                n = c < st.klen[b] ? min(st.W, st.klen[b] - c) : 0;
            }
        }
        const int act = n > 0;
        if (act) {
            atomicAdd(&sum_keys, c + n);
            atomicAdd(&sum_n, n);
        }
        // exclusive scan of act over the block
        int incl = act;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        int before = carry;
        for (int w = 0; w < wid; ++w) before += warp_tot[w];
        const int pos = before + incl - act;
        if (b < st.B) {
            if (compact) {
                if (act) {
                    st.slot_img[pos] = b;
                    st.slot_c[pos] = c;
                    st.slot_n[pos] = n;
                }
            } else {
                st.slot_img[b] = b;
                st.slot_c[b] = c;
                st.slot_n[b] = n;
            }
        }
        __syncthreads();
        if (tid == blockDim.x - 1) carry = before + incl;
        __syncthreads();
    }
    // slots by context length, longest first (ties by slot index): the attention kernel deals its work items
    // from this list so that every CTA streams about the same number of key blocks
    if (st.slot_order != nullptr) {
        __syncthreads();
        const int n_slots = compact ? carry : st.B;
        for (int s0 = tid; s0 < n_slots; s0 += blockDim.x) {
            const int len = st.slot_n[s0] > 0 ? st.slot_c[s0] + st.slot_n[s0] : -1;
            int rank = 0;
            for (int s1 = 0; s1 < n_slots; ++s1) {
                const int l1 = st.slot_n[s1] > 0 ? st.slot_c[s1] + st.slot_n[s1] : -1;
                rank += (l1 > len) || (l1 == len && s1 < s0);
            }
            st.slot_order[rank] = s0;
        }
    }
    if (tid == 0) {
        st.counters[CNT_LIVE_SETUP] = carry;
        st.counters[CNT_SLOTS] = compact ? carry : st.B;
        st.counters[CNT_LIVE] = 0;
        st.counters[CNT_SUM_KEYS] = sum_keys;
        st.counters[CNT_SUM_N] = sum_n;
    }
}

void launch_setup(const State& st, int phase, int compact, cudaStream_t s) {
    launch_k(k_setup, dim3(1), dim3(1024), 0, s, st, phase, compact);
}

__global__ void k_noop() {
    pdl_trigger();
    pdl_wait();
}
void launch_noop(cudaStream_t s) { launch_k(k_noop, dim3(1), dim3(32), 0, s); }

// ------------------------------------------------------------------ embedding gather
// hb / ssq (may be null): bf16 copy of the row and its sums of squares per 32-column chunk (what the RMSNorm
// folded into the first projection reads).  Warp w of the block owns chunks w, w + 4, ...; lane l element l.
template <typename TA>
__global__ void __launch_bounds__(128) k_embed(State st, int S, const TA* __restrict__ tok_emb,
                                               const TA* __restrict__ cls_emb, float* __restrict__ h,
                                               bf16* __restrict__ hb, float* __restrict__ ssq) {
    pdl_trigger();
    pdl_wait();
    const int row = blockIdx.x;
    const int i = row % st.W;
    const int slot = (row / st.W) % S;
    const int br = row / (st.W * S);
    const int n = st.slot_n[slot];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    float* dst = h + (size_t)row * st.D;
    const TA* src = nullptr;
    if (i < n) {
        const int img = st.slot_img[slot];
        const int s = st.slot_c[slot] + i;
        if (s == 0) {
            const int cls = br ? st.C : st.label[img];
            src = cls_emb + (size_t)cls * st.D;
        } else {
            src = tok_emb + (size_t)st.seq[(size_t)img * (st.T + 1) + s] * st.D;
        }
    }
    for (int chunk = wid; chunk * 32 < st.D; chunk += 4) {
        const int e = chunk * 32 + lane;
        const float v = (src != nullptr && e < st.D) ? to_f<TA>(src[e]) : 0.f;
        if (e < st.D) {
            dst[e] = v;
            if (hb != nullptr) hb[(size_t)row * st.D + e] = __float2bfloat16_rn(v);
        }
        if (ssq != nullptr) {
            const float ss = warp_sum(v * v);
            if (lane == 0) ssq[(size_t)row * (st.D / 32) + chunk] = ss;
        }
    }
}

template <typename TA>
void launch_embed(const State& st, int S, const TA* tok_emb, const TA* cls_emb, float* h, bf16* hb, float* ssq,
                  cudaStream_t s) {
    launch_k(k_embed<TA>, dim3(st.nb * S * st.W), dim3(128), 0, s, st, S, tok_emb, cls_emb, h, hb, ssq);
}
template void launch_embed<float>(const State&, int, const float*, const float*, float*, bf16*, float*, cudaStream_t);
template void launch_embed<bf16>(const State&, int, const bf16*, const bf16*, float*, bf16*, float*, cudaStream_t);

// ------------------------------------------------------------------ RMSNorm: out = x * rsqrt(mean(x^2)+eps) * g
// One warp per row; the row stays in registers between the two passes (D <= 2048 through the vector path).
// The sum of squares is reduced in a fixed order that depends on D only.
template <typename TA, int VEC_ITERS>
__global__ void __launch_bounds__(256) k_rmsnorm_warp(const float* __restrict__ h, const TA* __restrict__ gain,
                                                      TA* __restrict__ out, int M, int D, float eps) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= M) return;
    const float4* x4 = reinterpret_cast<const float4*>(h + (size_t)row * D);
    float4 v[VEC_ITERS];
    float ss = 0.f;
#pragma unroll
    for (int it = 0; it < VEC_ITERS; ++it) {
        const int idx = it * 32 + lane;
        if (idx * 4 < D) {
            v[it] = x4[idx];
            ss += v[it].x * v[it].x + v[it].y * v[it].y + v[it].z * v[it].z + v[it].w * v[it].w;
        }
    }
    ss = warp_sum(ss);
    const float r = 1.0f / sqrtf(ss / (float)D + eps);
    TA* o = out + (size_t)row * D;
#pragma unroll
    for (int it = 0; it < VEC_ITERS; ++it) {
        const int idx = it * 32 + lane;
        if (idx * 4 < D) {
            const int e = idx * 4;
            const float a = v[it].x * r * to_f<TA>(gain[e]), b = v[it].y * r * to_f<TA>(gain[e + 1]);
            const float c = v[it].z * r * to_f<TA>(gain[e + 2]), d = v[it].w * r * to_f<TA>(gain[e + 3]);
            if constexpr (sizeof(TA) == 2) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&lo);
                pk.y = *reinterpret_cast<uint32_t*>(&hi);
                *reinterpret_cast<uint2*>(o + e) = pk;
            } else {
                *reinterpret_cast<float4*>(o + e) = make_float4(a, b, c, d);
            }
        }
    }
}

template <typename TA>
__global__ void k_rmsnorm(const float* __restrict__ h, const TA* __restrict__ gain, TA* __restrict__ out, int D,
                          float eps) {
    pdl_trigger();
    pdl_wait();
    __shared__ float red[32];
    const int row = blockIdx.x;
    const float* x = h + (size_t)row * D;
    float ss = 0.f;
    for (int e = threadIdx.x; e < D; e += blockDim.x) ss += x[e] * x[e];
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) tot += red[w];
    const float r = 1.0f / sqrtf(tot / (float)D + eps);
    TA* o = out + (size_t)row * D;
    for (int e = threadIdx.x; e < D; e += blockDim.x) o[e] = from_f<TA>(x[e] * r * to_f<TA>(gain[e]));
}

template <typename TA>
void launch_rmsnorm(const float* h, const TA* gain, TA* out, int M, int D, float eps, cudaStream_t s) {
    if (D % 4 == 0 && D <= 2048) {
        const int grid = (M + 7) / 8;
        if (D <= 512) launch_k(k_rmsnorm_warp<TA, 4>, dim3(grid), dim3(256), 0, s, h, gain, out, M, D, eps);
        else if (D <= 1024) launch_k(k_rmsnorm_warp<TA, 8>, dim3(grid), dim3(256), 0, s, h, gain, out, M, D, eps);
        else launch_k(k_rmsnorm_warp<TA, 16>, dim3(grid), dim3(256), 0, s, h, gain, out, M, D, eps);
    } else {
        launch_k(k_rmsnorm<TA>, dim3(M), dim3(128), 0, s, h, gain, out, D, eps);
    }
}
template void launch_rmsnorm<float>(const float*, const float*, float*, int, int, float, cudaStream_t);
template void launch_rmsnorm<bf16>(const float*, const bf16*, bf16*, int, int, float, cudaStream_t);

// ------------------------------------------------------------------ 2D RoPE + KV write
// One thread per (row, rotation pair).  rope_cs: [T][dh/2][2] cos/sin by sequence index.
template <typename TA>
__global__ void k_rope_kv(State st, int S, int layer, const float* __restrict__ qkv,
                          const float* __restrict__ rope_cs, TA* __restrict__ q, KvView kv) {
    pdl_trigger();
    pdl_wait();
    const int row = blockIdx.x;
    const int i = row % st.W;
    const int slot = (row / st.W) % S;
    const int br = row / (st.W * S);
    const int n = st.slot_n[slot];
    const int D = st.D, half = st.dh / 2;
    TA* qo = q + (size_t)row * D;
    if (i >= n) {
        for (int pe = threadIdx.x; pe < D / 2; pe += blockDim.x) {
            qo[2 * pe] = from_f<TA>(0.f);
            qo[2 * pe + 1] = from_f<TA>(0.f);
        }
        return;
    }
    const int img = st.slot_img[slot];
    const int s = st.slot_c[slot] + i;
    const int crow = br * st.Bmax + img;
    const size_t off = kv.offset(layer, crow, s);
    TA* ko = (TA*)kv.k + off;
    TA* vo = (TA*)kv.v + off;
    const float* src = qkv + (size_t)row * 3 * D;
    for (int pe = threadIdx.x; pe < D / 2; pe += blockDim.x) {
        const int e = pe % half;
        const float cs = rope_cs[((size_t)s * half + e) * 2], sn = rope_cs[((size_t)s * half + e) * 2 + 1];
        const float qa = src[2 * pe], qb = src[2 * pe + 1];
        const float ka = src[D + 2 * pe], kb = src[D + 2 * pe + 1];
        qo[2 * pe] = from_f<TA>(qa * cs - qb * sn);
        qo[2 * pe + 1] = from_f<TA>(qa * sn + qb * cs);
        ko[2 * pe] = from_f<TA>(ka * cs - kb * sn);
        ko[2 * pe + 1] = from_f<TA>(ka * sn + kb * cs);
        vo[2 * pe] = from_f<TA>(src[2 * D + 2 * pe]);
        vo[2 * pe + 1] = from_f<TA>(src[2 * D + 2 * pe + 1]);
    }
}

template <typename TA>
void launch_rope_kv(const State& st, int S, int layer, const float* qkv, const float* rope_cs, TA* q, KvView kv,
                    cudaStream_t s) {
    launch_k(k_rope_kv<TA>, dim3(st.nb * S * st.W), dim3(128), 0, s, st, S, layer, qkv, rope_cs, q, kv);
}
template void launch_rope_kv<float>(const State&, int, int, const float*, const float*, float*, KvView, cudaStream_t);
template void launch_rope_kv<bf16>(const State&, int, int, const float*, const float*, bf16*, KvView, cudaStream_t);

// ------------------------------------------------------------------ reference attention (one warp per row, head)
// Query at sequence index s = c+i attends keys 0..s of its cache row (cached prefix + this round's
// window up to itself).  Two passes with the scores in shared memory; the reduction order depends on s only.
template <typename TA>
__global__ void k_attention_ref(State st, int S, int layer, const TA* __restrict__ q, KvView kv,
                                TA* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ float smem[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const int row = blockIdx.x;
    const int head = blockIdx.y * nw + wid;
    if (head >= st.Hh) return;
    const int i = row % st.W;
    const int slot = (row / st.W) % S;
    const int br = row / (st.W * S);
    const int n = st.slot_n[slot];
    const int dh = st.dh;
    TA* o = out + (size_t)row * st.D + head * dh;
    if (i >= n) {
        for (int e = lane; e < dh; e += 32) o[e] = from_f<TA>(0.f);
        return;
    }
    float* sc = smem + (size_t)wid * (st.T + dh);
    float* qs = sc + st.T;
    const int img = st.slot_img[slot];
    const int s = st.slot_c[slot] + i;
    const int crow = br * st.Bmax + img;
    const TA* qv = q + (size_t)row * st.D + head * dh;
    for (int e = lane; e < dh; e += 32) qs[e] = to_f<TA>(qv[e]);
    __syncwarp();
    const float scale = 1.0f / sqrtf((float)dh);
    float mx = -INFINITY;
    for (int t = lane; t <= s; t += 32) {
        const TA* k = (const TA*)kv.k + kv.offset(layer, crow, t) + head * dh;
        float dot = 0.f;
        for (int e = 0; e < dh; ++e) dot += qs[e] * to_f<TA>(k[e]);
        dot *= scale;
        sc[t] = dot;
        mx = fmaxf(mx, dot);
    }
    mx = warp_max(mx);
    float den = 0.f;
    for (int t = lane; t <= s; t += 32) {
        const float p = expf(sc[t] - mx);
        sc[t] = p;
        den += p;
    }
    den = warp_sum(den);
    __syncwarp();
    for (int e = lane; e < dh; e += 32) {
        float acc = 0.f;
        for (int t = 0; t <= s; ++t) {
            const TA* v = (const TA*)kv.v + kv.offset(layer, crow, t) + head * dh;
            acc += sc[t] * to_f<TA>(v[e]);
        }
        o[e] = from_f<TA>(acc / den);
    }
}

template <typename TA>
void launch_attention_ref(const State& st, int S, int layer, const TA* q, KvView kv, TA* out, cudaStream_t s) {
    const int nw = 4;
    dim3 grid(st.nb * S * st.W, (st.Hh + nw - 1) / nw);
    const size_t smem = (size_t)nw * (st.T + st.dh) * sizeof(float);
    launch_k(k_attention_ref<TA>, dim3(grid), dim3(nw * 32), smem, s, st, S, layer, q, kv, out);
}
template void launch_attention_ref<float>(const State&, int, int, const float*, KvView, float*, cudaStream_t);
template void launch_attention_ref<bf16>(const State&, int, int, const bf16*, KvView, bf16*, cudaStream_t);

// ------------------------------------------------------------------ SwiGLU: act = silu(gate) * up
template <typename TA>
__global__ void k_swiglu(const float* __restrict__ gu, TA* __restrict__ act, int F) {
    pdl_trigger();
    pdl_wait();
    const int row = blockIdx.y;
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= F) return;
    const float g = gu[(size_t)row * 2 * F + f], u = gu[(size_t)row * 2 * F + F + f];
    act[(size_t)row * F + f] = from_f<TA>(g / (1.0f + expf(-g)) * u);
}

template <typename TA>
void launch_swiglu(const float* gu, TA* act, int M, int F, cudaStream_t s) {
    dim3 grid((F + 255) / 256, M);
    launch_k(k_swiglu<TA>, dim3(grid), dim3(256), 0, s, gu, act, F);
}
template void launch_swiglu<float>(const float*, float*, int, int, cudaStream_t);
template void launch_swiglu<bf16>(const float*, bf16*, int, int, cudaStream_t);

// ------------------------------------------------------------------ CUDA-core GEMM (fp32 model; bf16 checker)
// C[M,N] (+)= A[M,K] . W[N,K]^T, fp32 accumulation in increasing k, 64x64 tile, 4x4 outputs per thread.
template <typename TA>
__global__ void __launch_bounds__(256) k_gemm_simt(const TA* __restrict__ A, const TA* __restrict__ W,
                                                   float* __restrict__ C, int M, int N, int K, int accumulate) {
    pdl_trigger();
    pdl_wait();
    __shared__ float As[16][64 + 4];
    __shared__ float Bs[16][64 + 4];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    for (int k0 = 0; k0 < K; k0 += 16) {
        for (int idx = threadIdx.x; idx < 64 * 16; idx += 256) {
            const int r = idx >> 4, kk = idx & 15;
            const int gm = m0 + r, gn = n0 + r, gk = k0 + kk;
            As[kk][r] = (gm < M && gk < K) ? to_f<TA>(A[(size_t)gm * K + gk]) : 0.f;
            Bs[kk][r] = (gn < N && gk < K) ? to_f<TA>(W[(size_t)gn * K + gk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                a[x] = As[kk][ty * 4 + x];
                b[x] = Bs[kk][tx * 4 + x];
            }
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int gm = m0 + ty * 4 + x;
        if (gm >= M) continue;
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int gn = n0 + tx * 4 + y;
            if (gn >= N) continue;
            float* c = C + (size_t)gm * N + gn;
            *c = accumulate ? (*c + acc[x][y]) : acc[x][y];
        }
    }
}

template <typename TA>
void launch_gemm_simt(const TA* A, const TA* W, float* C, int M, int N, int K, int accumulate, cudaStream_t s) {
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    launch_k(k_gemm_simt<TA>, dim3(grid), dim3(256), 0, s, A, W, C, M, N, K, accumulate);
}
template void launch_gemm_simt<float>(const float*, const float*, float*, int, int, int, int, cudaStream_t);
template void launch_gemm_simt<bf16>(const bf16*, const bf16*, float*, int, int, int, int, cudaStream_t);

}  // namespace hbsjd
