// Distillation score of completed trajectories (Eq. 3): the bidirectional KL between the student's and the
// teacher's next-token distributions at every generated position, reduced per image and over the batch.
//
// For p = softmax(s), q = softmax(t) the normalisers cancel in the symmetric sum:
//   D_biKL(p, q) = 1/2 KL(p || q) + 1/2 KL(q || p) = 1/2 sum_v (p_v - q_v) (s_v - t_v)
//               = 1/2 ( A / Z_s - B / Z_t ),   A = sum e^{s - m_s} (s - t), Z_s = sum e^{s - m_s},
//                                              B = sum e^{t - m_t} (s - t), Z_t = sum e^{t - m_t},
// so one pass over the two logit rows with running maxima is enough: 2 V floats read per position, one
// float written.  HBM-bound.
#include "internal.h"

namespace hbsjd {

namespace {

constexpr int BK_THREADS = 512;
constexpr int BK_WARPS = BK_THREADS / 32;

// Running (max, sum of exponentials, weighted sum) of one distribution.
struct Acc {
    float m, z, a;
};

__device__ __forceinline__ float rescale(float m_old, float m_new) {
    return m_old == -INFINITY ? 0.f : __expf(m_old - m_new);
}

__device__ __forceinline__ Acc merge(const Acc& x, const Acc& y) {
    Acc r;
    r.m = fmaxf(x.m, y.m);
    const float fx = rescale(x.m, r.m), fy = rescale(y.m, r.m);
    r.z = x.z * fx + y.z * fy;
    r.a = x.a * fx + y.a * fy;
    return r;
}

__device__ __forceinline__ Acc warp_merge(Acc x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Acc y;
        y.m = __shfl_xor_sync(0xffffffffu, x.m, o);
        y.z = __shfl_xor_sync(0xffffffffu, x.z, o);
        y.a = __shfl_xor_sync(0xffffffffu, x.a, o);
        x = merge(x, y);
    }
    return x;
}

// All threads of the CTA: D_biKL(softmax(s), softmax(t)) of one row pair; the result is valid in thread 0.
__device__ float bikl_row(const float* __restrict__ s, const float* __restrict__ t, int V) {
    __shared__ Acc red[2][BK_WARPS];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    Acc as = {-INFINITY, 0.f, 0.f}, at = {-INFINITY, 0.f, 0.f};
    // chunks of 4 float4 per thread and array: sixteen 16-byte loads in flight per thread
    for (int v0 = tid * 4; v0 < V; v0 += BK_THREADS * 4 * 4) {
        float4 x[4], y[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int v = v0 + k * BK_THREADS * 4;
            if (v < V) {
                x[k] = *reinterpret_cast<const float4*>(s + v);
                y[k] = *reinterpret_cast<const float4*>(t + v);
            } else {
                x[k] = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
                y[k] = x[k];
            }
        }
        float ms = as.m, mt = at.m;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            ms = fmaxf(ms, fmaxf(fmaxf(x[k].x, x[k].y), fmaxf(x[k].z, x[k].w)));
            mt = fmaxf(mt, fmaxf(fmaxf(y[k].x, y[k].y), fmaxf(y[k].z, y[k].w)));
        }
        const float fs = rescale(as.m, ms), ft = rescale(at.m, mt);
        as.m = ms;
        at.m = mt;
        as.z *= fs;
        as.a *= fs;
        at.z *= ft;
        at.a *= ft;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (v0 + k * BK_THREADS * 4 < V) {
                const float xs[4] = {x[k].x, x[k].y, x[k].z, x[k].w};
                const float ys[4] = {y[k].x, y[k].y, y[k].z, y[k].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float d = xs[e] - ys[e];
                    const float es = __expf(xs[e] - ms), et = __expf(ys[e] - mt);
                    as.z += es;
                    as.a = fmaf(es, d, as.a);
                    at.z += et;
                    at.a = fmaf(et, d, at.a);
                }
            }
        }
    }
    as = warp_merge(as);
    at = warp_merge(at);
    if (lane == 0) {
        red[0][wid] = as;
        red[1][wid] = at;
    }
    __syncthreads();
    float out = 0.f;
    if (tid == 0) {
        Acc rs = red[0][0], rt = red[1][0];
        for (int w = 1; w < BK_WARPS; ++w) {
            rs = merge(rs, red[0][w]);
            rt = merge(rt, red[1][w]);
        }
        out = 0.5f * (rs.a / rs.z - rt.a / rt.z);
    }
    return out;
}

__global__ void __launch_bounds__(BK_THREADS) k_bikl_rows(const float* __restrict__ ls, const float* __restrict__ lt,
                                                          int V, float* __restrict__ out) {
    pdl_trigger();
    pdl_wait();
    const size_t row = blockIdx.x;
    const float d = bikl_row(ls + row * V, lt + row * V, V);
    if (threadIdx.x == 0) out[row] = d;
}

// One CTA per (slot, input i) of a scoring chunk: input i of the slot is sequence index c + i, whose output
// is the distribution of position t = c + i + 1; the term counts when t > k (Eq. 3 sums t = k+1 .. T).
__global__ void __launch_bounds__(BK_THREADS) k_bikl_slots(State st, const float* __restrict__ ls,
                                                           const float* __restrict__ lt,
                                                           const int32_t* __restrict__ prefix_len,
                                                           float* __restrict__ pos) {
    pdl_trigger();
    pdl_wait();
    const int i = blockIdx.x, slot = blockIdx.y;
    if (i >= st.slot_n[slot]) return;
    const int img = st.slot_img[slot];
    const int idx = st.slot_c[slot] + i;
    if (idx < prefix_len[img]) return;
    const size_t row = (size_t)slot * st.W + i;
    const float d = bikl_row(ls + row * st.V, lt + row * st.V, st.V);
    if (threadIdx.x == 0) pos[(size_t)img * st.T + idx] = d;
}

// Trajectory state for scoring: every token of the completed sequence is an input (sequence indices
// 0..T-1 = class token, x_1..x_{T-1}), processed like a prefix of length T.
__global__ void k_score_init(State st, const int32_t* __restrict__ tokens, const int32_t* __restrict__ labels,
                             const int32_t* __restrict__ prefix_len, float* __restrict__ pos) {
    pdl_trigger();
    pdl_wait();
    const int b = blockIdx.x;
    int32_t* seq = st.seq + (size_t)b * (st.T + 1);
    uint8_t* dl = st.delta + (size_t)b * (st.T + 1);
    for (int t = threadIdx.x; t <= st.T; t += blockDim.x) {
        seq[t] = t >= 1 ? tokens[(size_t)b * st.T + t - 1] : 0;
        dl[t] = 0;
        if (pos && t < st.T) pos[(size_t)b * st.T + t] = 0.f;
    }
    if (threadIdx.x == 0) {
        st.cursor[b] = st.T;
        st.klen[b] = st.T;
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

// per_image[b] = (1 / (T - k_b)) sum_{t = k_b+1..T} pos[b][t-1]; *loss = mean over the images with k_b < T.
// One CTA; fixed summation order (lane-strided partial sums, shuffle tree, then images in index order).
__global__ void k_score_reduce(int B, int T, const int32_t* __restrict__ prefix_len, const float* __restrict__ pos,
                               float* __restrict__ per_image, float* __restrict__ loss) {
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (int b = wid; b < B; b += nw) {
        const int k = prefix_len[b];
        float acc = 0.f;
        for (int idx = k + lane; idx < T; idx += 32) acc += pos[(size_t)b * T + idx];
        acc = warp_sum(acc);
        if (lane == 0) per_image[b] = k < T ? acc / (float)(T - k) : 0.f;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
        int cnt = 0;
        for (int b = 0; b < B; ++b)
            if (prefix_len[b] < T) {
                tot += per_image[b];
                ++cnt;
            }
        *loss = cnt ? tot / (float)cnt : 0.f;
    }
}

}  // namespace

void launch_bikl_rows(const float* ls, const float* lt, int rows, int V, float* out, cudaStream_t s) {
    launch_k(k_bikl_rows, dim3(rows), dim3(BK_THREADS), 0, s, ls, lt, V, out);
}

void launch_bikl_slots(const State& st, int S, const float* ls, const float* lt, const int32_t* prefix_len,
                       float* pos, cudaStream_t s) {
    launch_k(k_bikl_slots, dim3(st.W, S), dim3(BK_THREADS), 0, s, st, ls, lt, prefix_len, pos);
}

void launch_score_init(const State& st, const int32_t* tokens, const int32_t* labels, const int32_t* prefix_len,
                       float* pos, cudaStream_t s) {
    launch_k(k_score_init, dim3(st.B), dim3(128), 0, s, st, tokens, labels, prefix_len, pos);
}

void launch_score_reduce(int B, int T, const int32_t* prefix_len, const float* pos, float* per_image, float* loss,
                         cudaStream_t s) {
    launch_k(k_score_reduce, dim3(1), dim3(1024), 0, s, B, T, prefix_len, pos, per_image, loss);
}

}  // namespace hbsjd
