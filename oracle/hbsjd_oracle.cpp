// CPU ORACLE for the HB-SJD rollout round.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, deliberately unoptimised restatement of what the rollout path
// computes, written from the paper's method section:
//   * the autoregressive factorisation that is being sampled        (Eq. 1, Eq. 2)
//   * independent per-image cursors and Jacobi windows               (Sec. 4.2, "Independent rollout states")
//   * one verifier forward over [last committed token | drafts]      (Sec. 4.2, "Batched verification")
//   * greedy verification                                            (Eq. 4)
//   * probabilistic SJD verification and residual resampling         (Eq. 5)
//   * independent progress, shared cond/uncond state under CFG,
//     replacement token = next start token, no cache repair          (Sec. 4.2, "Independent progress")
//   * Full / Compact / Hybrid execution choice                       (Sec. 4.3, Eq. 6)
//   * batch-synchronous progress, the baseline of the ablation        (Sec. 5.3, Table 2)
//   * the distillation score of a completed trajectory: teacher and
//     student full-sequence forwards and the bidirectional KL          (Eq. 3)
//
// Only tests, the smoke check and the benchmark's cpu_baseline leg may call
// this file.  It shares no code, header, table or constant generator with the
// CUDA library; the product never links or imports it.
//
// Arithmetic: weights exactly as stored (bf16 widened, or fp32); every dot
// product, norm, softmax and rotation accumulates in double; activations are
// stored as fp32.  When `act_bf16` is set (bf16 model), the operand of every
// matrix product, the rotated q/k and v (the KV-cache contents) and the
// attention output are rounded to bf16 (round-to-nearest-even) at exactly the
// points listed in forward_window() below.  Each (image, position) is
// computed in an order that does not depend on batch or window shape.
//
// Pins (tests/test_oracle_*.py): Philox known answers; forward against an
// independent fp64 torch restatement; cached window forward == full recompute;
// RoPE shift invariance; softmax/top-k properties; W=1 rollout == plain AR
// sampler; greedy SJD == greedy AR; accept/resample identity by brute force;
// chi-square of SJD rollouts against the enumerated AR joint; Full == Compact;
// subset independence; CFG special cases; batch-synchronous progress (common
// pace, truncation by hand, greedy exactness, chi-square of batches of three);
// bidirectional KL closed forms (two
// classes, equal distributions, shift invariance, symmetry) and the score
// against the torch restatement's logits.
// Parity unpinned: the absolute token values for a given seed (the paper
// prints no worked example).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ------------------------------------------------------------------ helpers

inline float bf16_round(float x) {
    uint32_t u;
    std::memcpy(&u, &x, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return x;  // NaN passes through
    uint32_t r = u + 0x7fffu + ((u >> 16) & 1u);
    r &= 0xffff0000u;
    float y;
    std::memcpy(&y, &r, 4);
    return y;
}

inline float bf16_widen(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float y;
    std::memcpy(&y, &u, 4);
    return y;
}

// Philox4x32-10 (Salmon et al., SC'11).
void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

struct Desc {
    int32_t L, D, Hh, F, V, gh, gw, C, dtype;  // dtype 0 = fp32, 1 = bf16
    float eps, rope_base;
};

struct Layer {
    std::vector<float> g_attn, w_qkv, w_o, g_ffn, w_13, w_2;
};

struct Model {
    Desc d;
    int T, dh;
    int act_bf16;
    // Diagnostics only (noise-floor calibration; never a comparison target):
    int acc_f32 = 0;      // dot products and sums of squares accumulate in fp32 instead of double
    int attn_w_bf16 = 0;  // the unnormalised attention weights are rounded to bf16 before they multiply the values
                          // (the usual tensor-core formulation; the normaliser keeps the unrounded weights)
    int norm_folded = 0;  // RMSNorm(x) W^T evaluated as r (bf16(x) diag(g) W^T), r = rsqrt(mean(x^2) + eps): the row
                          // factor applied after the product instead of before it (the same function of x)
    std::vector<float> tok_emb, cls_emb, g_out, w_head;
    std::vector<Layer> layers;
};

size_t load_tensor(const Desc& d, const uint8_t* img, size_t off, size_t count, std::vector<float>& dst) {
    dst.resize(count);
    if (d.dtype == 0) {
        std::memcpy(dst.data(), img + off, count * 4);
        off += count * 4;
    } else {
        const uint16_t* p = (const uint16_t*)(img + off);
        for (size_t i = 0; i < count; ++i) dst[i] = bf16_widen(p[i]);
        off += count * 2;
    }
    return (off + 255) / 256 * 256;
}

// Y[n][N] = X[n][K] . W[N][K]^T, every output a sum over k in increasing k, accumulated in Acc (double; float
// only for the noise-floor diagnostic).  Output columns are spread over the host threads unless the caller already
// runs one image per thread; an output's own sum is the same either way.
template <typename Acc>
void matmul_acc(const float* X, int n, int K, const float* W, int N, float* Y) {
    std::vector<Acc> Xt((size_t)K * n);
    for (int i = 0; i < n; ++i)
        for (int k = 0; k < K; ++k) Xt[(size_t)k * n + i] = (Acc)X[(size_t)i * K + k];
#pragma omp parallel for schedule(static) if (!omp_in_parallel() && (size_t)N * K * n > 200000)
    for (int o = 0; o < N; ++o) {
        std::vector<Acc> acc(n, (Acc)0);
        const float* w = W + (size_t)o * K;
        for (int k = 0; k < K; ++k) {
            const Acc wk = (Acc)w[k];
            const Acc* xr = &Xt[(size_t)k * n];
            for (int i = 0; i < n; ++i) acc[i] += wk * xr[i];
        }
        for (int i = 0; i < n; ++i) Y[(size_t)i * N + o] = (float)acc[i];
    }
}

void matmul(const Model& M, const float* X, int n, int K, const float* W, int N, float* Y) {
    if (M.acc_f32) matmul_acc<float>(X, n, K, W, N, Y);
    else matmul_acc<double>(X, n, K, W, N, Y);
}

// out = x * rsqrt(mean(x^2) + eps) * g
void rmsnorm(const Model& M, const float* x, const float* g, float* out) {
    const int D = M.d.D;
    double ss = 0.0;
    if (M.acc_f32) {
        float sf = 0.0f;
        for (int k = 0; k < D; ++k) sf += x[k] * x[k];
        ss = sf;
    } else {
        for (int k = 0; k < D; ++k) ss += (double)x[k] * x[k];
    }
    const double r = 1.0 / std::sqrt(ss / D + (double)M.d.eps);
    for (int k = 0; k < D; ++k) {
        float v = (float)((double)x[k] * r * (double)g[k]);
        out[k] = M.act_bf16 ? bf16_round(v) : v;
    }
}

inline float maybe_bf16(const Model& M, float v) { return M.act_bf16 ? bf16_round(v) : v; }

// Y[n][N] = RMSNorm(x; g) W^T for n rows; a[n][D] receives the operand of the product.  The definition (norm, round
// the operand, multiply) unless the diagnostic norm_folded is set.
void normed_projection(const Model& M, const float* x, const float* g, int n, const float* W, int N, float* a,
                       float* Y) {
    const int D = M.d.D;
    if (!M.norm_folded) {
        for (int i = 0; i < n; ++i) rmsnorm(M, &x[(size_t)i * D], g, &a[(size_t)i * D]);
        matmul(M, a, n, D, W, N, Y);
        return;
    }
    std::vector<double> r(n);
    for (int i = 0; i < n; ++i) {
        double ss = 0.0;
        for (int k = 0; k < D; ++k) ss += (double)x[(size_t)i * D + k] * x[(size_t)i * D + k];
        r[i] = 1.0 / std::sqrt(ss / D + (double)M.d.eps);
        for (int k = 0; k < D; ++k) a[(size_t)i * D + k] = maybe_bf16(M, x[(size_t)i * D + k]) * g[k];
    }
    matmul(M, a, n, D, W, N, Y);
    for (int i = 0; i < n; ++i)
        for (int o = 0; o < N; ++o) Y[(size_t)i * N + o] = (float)((double)Y[(size_t)i * N + o] * r[i]);
}

// 2D rotary embedding on one head vector at sequence index s.
// Index 0 (class token) is not rotated.  Index s >= 1 is image token s-1 at
// (row, col) = ((s-1) / gw, (s-1) % gw).  Adjacent pairs (2e, 2e+1): the first
// dh/4 pairs turn by row * w_e, the other dh/4 by col * w_e, w_e = base^(-e/(dh/4)).
void rope2d(const Model& M, float* v, int s) {
    if (s == 0) return;
    const int dh = M.dh, quarter = dh / 4;
    const int row = (s - 1) / M.d.gw, col = (s - 1) % M.d.gw;
    for (int e = 0; e < dh / 2; ++e) {
        const int ee = e < quarter ? e : e - quarter;
        const double pos = e < quarter ? (double)row : (double)col;
        const double w = std::pow((double)M.d.rope_base, -(double)ee / (double)quarter);
        const double ang = pos * w;
        const double cs = std::cos(ang), sn = std::sin(ang);
        const double a = v[2 * e], b = v[2 * e + 1];
        v[2 * e] = (float)(a * cs - b * sn);
        v[2 * e + 1] = (float)(a * sn + b * cs);
    }
}

void embed(const Model& M, int label, const int32_t* seq, int s, float* x) {
    const int D = M.d.D;
    const float* e = (s == 0) ? &M.cls_emb[(size_t)label * D] : &M.tok_emb[(size_t)seq[s] * D];
    for (int k = 0; k < D; ++k) x[k] = e[k];
}

// Copies of one layer's intermediates of forward_window, for component parity tests (any pointer may be null).
// Row i belongs to sequence index c + i.
struct Trace {
    int32_t layer;
    float* a;       // [n][D]  normed input of the QKV projection
    float* q;       // [n][D]  rotated queries
    float* k;       // [n][D]  rotated keys as cached
    float* v;       // [n][D]  values as cached
    float* o;       // [n][D]  attention output
    float* x_attn;  // [n][D]  residual stream after the attention sub-block
    float* m;       // [n][D]  normed input of the gate/up projection
    float* act;     // [n][F]  silu(gate) * up
    float* x_out;   // [n][D]  residual stream after the block
};

inline void trace_copy(float* dst, const float* src, size_t count) {
    if (dst) std::memcpy(dst, src, count * sizeof(float));
}

// FFN sub-block in two stages: m = RMSNorm(x; g_ffn) (bf16), act = silu(W1 m) * (W3 m) (bf16); x += W2 act.
void stage_ffn_act(const Model& M, const Layer& Ly, const float* x, int n, float* m, float* act) {
    const int D = M.d.D, F = M.d.F;
    std::vector<float> gu((size_t)n * 2 * F);
    normed_projection(M, x, Ly.g_ffn.data(), n, Ly.w_13.data(), 2 * F, m, gu.data());
    for (int i = 0; i < n; ++i)
        for (int f = 0; f < F; ++f) {
            const double g = gu[(size_t)i * 2 * F + f], u = gu[(size_t)i * 2 * F + F + f];
            const double silu = g / (1.0 + std::exp(-g));
            act[(size_t)i * F + f] = maybe_bf16(M, (float)(silu * u));
        }
}

void stage_ffn_down(const Model& M, const Layer& Ly, const float* act, int n, float* x) {
    const int D = M.d.D, F = M.d.F;
    std::vector<float> y((size_t)n * D);
    matmul(M, act, n, F, Ly.w_2.data(), D, y.data());
    for (size_t k = 0; k < (size_t)n * D; ++k) x[k] = x[k] + y[k];
}

void ffn_block(const Model& M, const Layer& Ly, std::vector<float>& x, int n, const Trace* tr = nullptr) {
    const int D = M.d.D, F = M.d.F;
    std::vector<float> m((size_t)n * D), act((size_t)n * F);
    stage_ffn_act(M, Ly, x.data(), n, m.data(), act.data());
    stage_ffn_down(M, Ly, act.data(), n, x.data());
    if (tr) {
        trace_copy(tr->m, m.data(), (size_t)n * D);
        trace_copy(tr->act, act.data(), (size_t)n * F);
        trace_copy(tr->x_out, x.data(), (size_t)n * D);
    }
}

void head(const Model& M, const std::vector<float>& x, int n, float* logits) {
    const int D = M.d.D;
    std::vector<float> hn((size_t)n * D);
    normed_projection(M, x.data(), M.g_out.data(), n, M.w_head.data(), M.d.V, hn.data(), logits);
}

// Attention of one query vector q (head h) at sequence index s over keys 0..s
// read from K,V laid out [idx][D].
void attend(const Model& M, const float* q, const float* K, const float* V, int h, int s, float* out) {
    const int D = M.d.D, dh = M.dh;
    const double scale = 1.0 / std::sqrt((double)dh);
    std::vector<double> sc(s + 1);
    double mx = -1e300;
    for (int t = 0; t <= s; ++t) {
        const float* k = K + (size_t)t * D + h * dh;
        double dot = 0.0;
        if (M.acc_f32) {
            float df = 0.0f;
            for (int e = 0; e < dh; ++e) df += q[e] * k[e];
            dot = df;
        } else {
            for (int e = 0; e < dh; ++e) dot += (double)q[e] * (double)k[e];
        }
        sc[t] = dot * scale;
        mx = std::max(mx, sc[t]);
    }
    double den = 0.0;
    for (int t = 0; t <= s; ++t) {
        sc[t] = std::exp(sc[t] - mx);
        den += sc[t];
        if (M.attn_w_bf16) sc[t] = bf16_round((float)sc[t]);
    }
    for (int e = 0; e < dh; ++e) {
        double acc = 0.0;
        if (M.acc_f32) {
            float af = 0.0f;
            for (int t = 0; t <= s; ++t) af += (float)sc[t] * V[(size_t)t * D + h * dh + e];
            acc = af;
        } else {
            for (int t = 0; t <= s; ++t) acc += sc[t] * (double)V[(size_t)t * D + h * dh + e];
        }
        out[e] = maybe_bf16(M, (float)(acc / den));
    }
}

// Attention sub-block in three stages, rows i = 0..n-1 at sequence indices c+i.
// (1) a = RMSNorm(x; g_attn) (bf16); qkv[i] = [q | k | v] = W_qkv a, q and k rotated by the 2D RoPE of index
//     c+i, all three rounded (bf16): q is the query operand, k and v are the cache contents.
void stage_qkv(const Model& M, const Layer& Ly, const float* x, int n, int c, float* a, float* qkv) {
    const int D = M.d.D, dh = M.dh, Hh = M.d.Hh;
    normed_projection(M, x, Ly.g_attn.data(), n, Ly.w_qkv.data(), 3 * D, a, qkv);  // a: (bf16)
    for (int i = 0; i < n; ++i) {
        float* q = &qkv[(size_t)i * 3 * D];
        float* k = q + D;
        for (int h = 0; h < Hh; ++h) {
            rope2d(M, q + h * dh, c + i);
            rope2d(M, k + h * dh, c + i);
        }
        for (int e = 0; e < 3 * D; ++e) q[e] = maybe_bf16(M, q[e]);  // (bf16) query operand, cache contents
    }
}

// (2) o[i] = causal attention of query i (row stride ldq) over keys 0..c+i of K, V laid out [idx][D]   (bf16)
void stage_attend(const Model& M, const float* q, size_t ldq, const float* Kl, const float* Vl, int c, int n,
                  float* o) {
    const int D = M.d.D, dh = M.dh, Hh = M.d.Hh;
    for (int i = 0; i < n; ++i)
        for (int h = 0; h < Hh; ++h)
            attend(M, q + (size_t)i * ldq + h * dh, Kl, Vl, h, c + i, &o[(size_t)i * D + h * dh]);
}

// (3) x += W_o o
void stage_attn_out(const Model& M, const Layer& Ly, const float* o, int n, float* x) {
    const int D = M.d.D;
    std::vector<float> y((size_t)n * D);
    matmul(M, o, n, D, Ly.w_o.data(), D, y.data());
    for (size_t k = 0; k < (size_t)n * D; ++k) x[k] = x[k] + y[k];
}

// Windowed forward with a per-row KV cache (Sec. 4.2, "Batched verification").
// Inputs: sequence indices c .. c+n-1 of one physical row (index 0 = class
// token `label`, index s >= 1 = token seq[s]).  kc/vc are [L][T][D]; entries
// 0..c-1 must be valid; entries c..c+n-1 are (over)written.  If logits != null
// it receives [n][V] (position i predicts the token at sequence index c+i+1).
void forward_window(const Model& M, float* kc, float* vc, int label, const int32_t* seq, int c, int n,
                    float* logits, const Trace* trace = nullptr) {
    const int D = M.d.D, T = M.T;
    std::vector<float> x((size_t)n * D), a((size_t)n * D), qkv((size_t)n * 3 * D), o((size_t)n * D);
    for (int i = 0; i < n; ++i) embed(M, label, seq, c + i, &x[(size_t)i * D]);
    for (int l = 0; l < M.d.L; ++l) {
        const Layer& Ly = M.layers[l];
        float* Kl = kc + (size_t)l * T * D;
        float* Vl = vc + (size_t)l * T * D;
        stage_qkv(M, Ly, x.data(), n, c, a.data(), qkv.data());
        for (int i = 0; i < n; ++i) {  // the window's keys and values enter the cache before attention reads it
            std::memcpy(Kl + (size_t)(c + i) * D, &qkv[(size_t)i * 3 * D + D], D * sizeof(float));
            std::memcpy(Vl + (size_t)(c + i) * D, &qkv[(size_t)i * 3 * D + 2 * D], D * sizeof(float));
        }
        stage_attend(M, qkv.data(), (size_t)3 * D, Kl, Vl, c, n, o.data());
        stage_attn_out(M, Ly, o.data(), n, x.data());
        const Trace* tr = (trace && trace->layer == l) ? trace : nullptr;
        if (tr) {
            trace_copy(tr->a, a.data(), (size_t)n * D);
            for (int i = 0; i < n; ++i) {
                if (tr->q) std::memcpy(tr->q + (size_t)i * D, &qkv[(size_t)i * 3 * D], D * sizeof(float));
                if (tr->k) std::memcpy(tr->k + (size_t)i * D, Kl + (size_t)(c + i) * D, D * sizeof(float));
                if (tr->v) std::memcpy(tr->v + (size_t)i * D, Vl + (size_t)(c + i) * D, D * sizeof(float));
            }
            trace_copy(tr->o, o.data(), (size_t)n * D);
            trace_copy(tr->x_attn, x.data(), (size_t)n * D);
        }
        ffn_block(M, Ly, x, n, tr);
    }
    if (logits) head(M, x, n, logits);
}

// Full-recompute forward of one sequence of `len` indices (no cache object):
// textbook causal attention over the whole sequence.  logits: [len][V].
void forward_full(const Model& M, int label, const int32_t* seq, int len, float* logits) {
    const int D = M.d.D, dh = M.dh, Hh = M.d.Hh;
    std::vector<float> x((size_t)len * D), a((size_t)len * D), qkv((size_t)len * 3 * D), o((size_t)len * D),
        y((size_t)len * D), K((size_t)len * D), V((size_t)len * D);
    for (int s = 0; s < len; ++s) embed(M, label, seq, s, &x[(size_t)s * D]);
    for (int l = 0; l < M.d.L; ++l) {
        const Layer& Ly = M.layers[l];
        for (int s = 0; s < len; ++s) rmsnorm(M, &x[(size_t)s * D], Ly.g_attn.data(), &a[(size_t)s * D]);
        matmul(M, a.data(), len, D, Ly.w_qkv.data(), 3 * D, qkv.data());
        for (int s = 0; s < len; ++s) {
            float* q = &qkv[(size_t)s * 3 * D];
            for (int h = 0; h < Hh; ++h) {
                rope2d(M, q + h * dh, s);
                rope2d(M, q + D + h * dh, s);
            }
            for (int e = 0; e < D; ++e) {
                q[e] = maybe_bf16(M, q[e]);
                K[(size_t)s * D + e] = maybe_bf16(M, q[D + e]);
                V[(size_t)s * D + e] = maybe_bf16(M, q[2 * D + e]);
            }
        }
        for (int s = 0; s < len; ++s)
            for (int h = 0; h < Hh; ++h)
                attend(M, &qkv[(size_t)s * 3 * D + h * dh], K.data(), V.data(), h, s, &o[(size_t)s * D + h * dh]);
        matmul(M, o.data(), len, D, Ly.w_o.data(), D, y.data());
        for (size_t k = 0; k < (size_t)len * D; ++k) x[k] = x[k] + y[k];
        ffn_block(M, Ly, x, len);
    }
    head(M, x, len, logits);
}

// ------------------------------------------------------- probability pipeline

// Guided logits -> temperature -> top-k (ties at the k-th value all kept) ->
// softmax, rounded to fp32.  lu == null or s == 1: no guidance ("fused guided
// logits", Sec. 4.2 "Independent progress").
void probs(const float* lc, const float* lu, float s, float tau, int k, int V, float* p) {
    std::vector<float> g(V);
    for (int v = 0; v < V; ++v) {
        float x = lc[v];
        if (lu) x = (float)((double)lu[v] + (double)s * ((double)lc[v] - (double)lu[v]));
        g[v] = (float)((double)x / (double)tau);
    }
    float theta = -INFINITY;
    if (k > 0 && k < V) {
        std::vector<float> srt(g);
        std::nth_element(srt.begin(), srt.begin() + (k - 1), srt.end(), [](float a, float b) { return a > b; });
        theta = srt[k - 1];
    }
    double mx = -1e300;
    for (int v = 0; v < V; ++v)
        if (g[v] >= theta) mx = std::max(mx, (double)g[v]);
    std::vector<double> e(V);
    double den = 0.0;
    for (int v = 0; v < V; ++v) {
        e[v] = (g[v] >= theta) ? std::exp((double)g[v] - mx) : 0.0;
        den += e[v];
    }
    for (int v = 0; v < V; ++v) p[v] = (float)(e[v] / den);
}

// Fixed-point categorical sample: w_v = floor(a_v * 2^30); S = sum w; target =
// (word * S) >> 32; smallest v whose inclusive running sum exceeds target.
// Returns -1 when S == 0.
int sample_fixed(const float* a, int V, uint32_t word) {
    uint64_t S = 0;
    for (int v = 0; v < V; ++v) S += (uint64_t)(uint32_t)std::floor(a[v] * 1073741824.0f);
    if (S == 0) return -1;
    const uint64_t target = ((uint64_t)word * S) >> 32;
    uint64_t run = 0;
    for (int v = 0; v < V; ++v) {
        run += (uint64_t)(uint32_t)std::floor(a[v] * 1073741824.0f);
        if (run > target) return v;
    }
    return V - 1;  // unreachable
}

int argmax_low(const float* p, int V) {
    int best = 0;
    for (int v = 1; v < V; ++v)
        if (p[v] > p[best]) best = v;
    return best;
}

struct Params {
    int32_t window, history, top_k, verify_mode /*0 prob, 1 greedy*/,
        exec_mode /*0 full, 1 compact, 2 hybrid, 3 full with batch-synchronous progress*/, gamma;
    float cfg_scale, temperature;
    uint64_t seed;
};

// Verification, commit and draft refresh of one image for one round, given
// this round's probabilities (Eq. 4 / Eq. 5; Sec. 4.2 "Independent rollout
// states" for the refresh).  words[i] are the four random words of token
// position t = c+i+1; w3_beyond[d] is word 3 of position c+n+1+d.
//   p     [n][V]   p[i] = distribution of token c+i+1
//   qprev          previous round's probabilities; the proposal of the draft at
//                  position t is row (t - qbase - 1)
// Returns m (tokens committed) and the first-reject index in *j_out (-1: none).
// Index of the first rejected draft of the window (Eq. 4 / Eq. 5), -1 if every draft is accepted.
int first_reject(int V, bool greedy, int c, const int32_t* seq, const uint8_t* delta, const float* p, int n,
                 const float* qprev, int qbase, const uint32_t (*words)[4]) {
    int j = -1;
    for (int i = 0; i + 1 < n; ++i) {
        const int t = c + i + 1;
        const int z = seq[t];
        bool accept;
        if (greedy) {
            accept = (z == argmax_low(p + (size_t)i * V, V));
        } else {
            const float pz = p[(size_t)i * V + z];
            float alpha;
            if (delta[t]) {
                alpha = pz;  // point-mass proposal
            } else {
                const float qz = qprev[(size_t)(t - qbase - 1) * V + z];
                alpha = std::min(1.0f, pz / qz);
            }
            const float u = (float)(words[i][0] >> 8) * (1.0f / 16777216.0f);
            accept = u < alpha;
        }
        if (!accept) { j = i; break; }
    }
    return j;
}

// m_limit > 0 (batch-synchronous progress, the baseline of Sec. 5.3 "Is independent progress necessary"):
// commit at most m_limit tokens.  An image whose own verification would commit more keeps only the first
// m_limit of its accepted drafts (no replacement token is drawn: every one of them was accepted); *j_out is
// then -1.
int decide_and_refresh(int V, int T, int W, int H, bool greedy, int& c, int32_t* seq, uint8_t* delta,
                       const float* p, int n, const float* qprev, int qbase, const uint32_t (*words)[4],
                       const uint32_t* w3_beyond, int* j_out, int m_limit = 0) {
    int j = first_reject(V, greedy, c, seq, delta, p, n, qprev, qbase, words);
    int m, tok;
    if (m_limit > 0 && m_limit < (j >= 0 ? j + 1 : n)) {
        m = m_limit;
        tok = seq[c + m];  // an accepted draft
        j = -1;
    } else if (j >= 0) {
        const int t = c + j + 1;
        const float* pj = p + (size_t)j * V;
        if (greedy) {
            tok = argmax_low(pj, V);
        } else {
            std::vector<float> r(V);
            if (delta[t]) {
                for (int v = 0; v < V; ++v) r[v] = pj[v];
                r[seq[t]] = 0.0f;
            } else {
                const float* q = qprev + (size_t)(t - qbase - 1) * V;
                for (int v = 0; v < V; ++v) {
                    const float d = pj[v] - q[v];
                    r[v] = d > 0.0f ? d : 0.0f;
                }
            }
            tok = sample_fixed(r.data(), V, words[j][1]);
            if (tok < 0) tok = sample_fixed(pj, V, words[j][1]);
        }
        m = j + 1;
    } else {
        const float* pl = p + (size_t)(n - 1) * V;
        tok = greedy ? argmax_low(pl, V) : sample_fixed(pl, V, words[n - 1][1]);
        m = n;
    }
    const int c_old = c;
    seq[c_old + m] = tok;
    delta[c_old + m] = 0;
    c = c_old + m;
    if (c < T) {
        const int n2 = std::min(W, T - c);
        for (int t = c + 1; t <= c + n2 - 1; ++t) {
            if (t <= c_old + n) {
                const int i = t - c_old - 1;
                const float* pi = p + (size_t)i * V;
                seq[t] = greedy ? argmax_low(pi, V) : sample_fixed(pi, V, words[i][2]);
                delta[t] = 0;
            } else {
                const int src = t - H;
                if (src >= 1) seq[t] = seq[src];
                else seq[t] = (int32_t)(((uint64_t)w3_beyond[t - (c_old + n) - 1] * (uint64_t)V) >> 32);
                delta[t] = 1;
            }
        }
    }
    *j_out = j;
    return m;
}

struct Image {
    int id, label, k, c, qbase;
    std::vector<int32_t> seq;    // [T+1], seq[t] = token x_t (1-based), seq[0] unused
    std::vector<uint8_t> delta;  // [T+1]
    std::vector<float> kc, vc, ku, vu;  // [L][T][D] conditional / unconditional caches
    std::vector<float> pcur, pprev;     // [W][V]
    std::vector<float> logc, logu;      // last round's logits [W][V]
    int last_n = 0;
};

struct Rollout {
    const Model* M;
    Params P;
    int B, round;
    std::vector<Image> img;
    std::vector<int32_t> trace_live, trace_mode;  // per executed round: A^(r) and 0 = Full / 1 = Compact
    long long image_forwards = 0, committed = 0, rejects = 0;
};

void words_for(const Params& P, int id, int t, uint32_t r, uint32_t out[4]) {
    const uint32_t ctr[4] = {(uint32_t)id, (uint32_t)t, r, 0u};
    const uint32_t key[2] = {(uint32_t)(P.seed & 0xffffffffu), (uint32_t)(P.seed >> 32)};
    philox4x32_10(ctr, key, out);
}

void init_window(const Rollout& R, Image& im) {
    const Model& M = *R.M;
    const int T = M.T, W = R.P.window, H = R.P.history;
    if (im.c >= T) return;
    const int n = std::min(W, T - im.c);
    for (int t = im.c + 1; t <= im.c + n - 1; ++t) {
        const int src = t - H;
        if (src >= 1) im.seq[t] = im.seq[src];
        else {
            uint32_t w[4];
            words_for(R.P, im.id, t, 0xFFFFFFFFu, w);
            im.seq[t] = (int32_t)(((uint64_t)w[3] * (uint64_t)M.d.V) >> 32);
        }
        im.delta[t] = 1;
    }
}

// Prefix pre-filling: cache sequence indices 0..k-1 (class token and the first
// k-1 prefix tokens) in chunks of W; no logits needed.
void prefill(const Rollout& R, Image& im) {
    const Model& M = *R.M;
    const bool cfg = R.P.cfg_scale != 1.0f;
    for (int pc = 0; pc < im.k; pc += R.P.window) {
        const int n = std::min(R.P.window, im.k - pc);
        forward_window(M, im.kc.data(), im.vc.data(), im.label, im.seq.data(), pc, n, nullptr);
        if (cfg) forward_window(M, im.ku.data(), im.vu.data(), M.d.C, im.seq.data(), pc, n, nullptr);
    }
}

// Forward of the image's window and this round's probabilities (left in im.pcur).
void image_forward(Rollout& R, Image& im) {
    const Model& M = *R.M;
    const int T = M.T, V = M.d.V, W = R.P.window;
    const bool cfg = R.P.cfg_scale != 1.0f;
    const int n = std::min(W, T - im.c);
    forward_window(M, im.kc.data(), im.vc.data(), im.label, im.seq.data(), im.c, n, im.logc.data());
    if (cfg) forward_window(M, im.ku.data(), im.vu.data(), M.d.C, im.seq.data(), im.c, n, im.logu.data());
    for (int i = 0; i < n; ++i)
        probs(&im.logc[(size_t)i * V], cfg ? &im.logu[(size_t)i * V] : nullptr, R.P.cfg_scale, R.P.temperature,
              R.P.top_k, V, &im.pcur[(size_t)i * V]);
}

void image_words(const Rollout& R, const Image& im, int n, std::vector<uint32_t>& words, std::vector<uint32_t>& beyond) {
    const int W = R.P.window;
    words.resize((size_t)n * 4);
    beyond.resize(W);
    for (int i = 0; i < n; ++i) words_for(R.P, im.id, im.c + i + 1, (uint32_t)R.round, &words[(size_t)i * 4]);
    for (int d = 0; d < W; ++d) {
        uint32_t w[4];
        words_for(R.P, im.id, im.c + n + 1 + d, (uint32_t)R.round, w);
        beyond[d] = w[3];
    }
}

// Tokens the image's own verification would commit this round (after image_forward).
int image_natural_commit(const Rollout& R, const Image& im) {
    const int T = R.M->T, V = R.M->d.V;
    const int n = std::min(R.P.window, T - im.c);
    std::vector<uint32_t> words, beyond;
    image_words(R, im, n, words, beyond);
    const int j = first_reject(V, R.P.verify_mode == 1, im.c, im.seq.data(), im.delta.data(), im.pcur.data(), n,
                               im.pprev.data(), im.qbase, (const uint32_t (*)[4])words.data());
    return j >= 0 ? j + 1 : n;
}

// Verification, commit and refresh after image_forward; m_limit as in decide_and_refresh.
int image_commit(Rollout& R, Image& im, int* j_out, int m_limit) {
    const int T = R.M->T, V = R.M->d.V, W = R.P.window;
    const int n = std::min(W, T - im.c);
    std::vector<uint32_t> words, beyond;
    image_words(R, im, n, words, beyond);
    const int c_old = im.c;
    const int m = decide_and_refresh(V, T, W, R.P.history, R.P.verify_mode == 1, im.c, im.seq.data(), im.delta.data(),
                                     im.pcur.data(), n, im.pprev.data(), im.qbase,
                                     (const uint32_t (*)[4])words.data(), beyond.data(), j_out, m_limit);
    im.pprev.swap(im.pcur);
    im.qbase = c_old;
    im.last_n = n;
    return m;
}

int image_round(Rollout& R, Image& im, int* j_out) {
    image_forward(R, im);
    return image_commit(R, im, j_out, 0);
}

}  // namespace

// ------------------------------------------------------------------- C entry

extern "C" {

void orc_philox(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox4x32_10(ctr, key, out); }

float orc_bf16_round(float x) { return bf16_round(x); }

void* orc_model_create(const Desc* d, const void* weights, size_t bytes, int act_bf16) {
    Model* M = new Model();
    M->d = *d;
    M->T = d->gh * d->gw;
    M->dh = d->D / d->Hh;
    M->act_bf16 = act_bf16;
    const uint8_t* img = (const uint8_t*)weights;
    const size_t D = d->D, F = d->F, V = d->V;
    size_t off = 0;
    off = load_tensor(*d, img, off, V * D, M->tok_emb);
    off = load_tensor(*d, img, off, (size_t)(d->C + 1) * D, M->cls_emb);
    M->layers.resize(d->L);
    for (int l = 0; l < d->L; ++l) {
        Layer& Ly = M->layers[l];
        off = load_tensor(*d, img, off, D, Ly.g_attn);
        off = load_tensor(*d, img, off, 3 * D * D, Ly.w_qkv);
        off = load_tensor(*d, img, off, D * D, Ly.w_o);
        off = load_tensor(*d, img, off, D, Ly.g_ffn);
        off = load_tensor(*d, img, off, 2 * F * D, Ly.w_13);
        off = load_tensor(*d, img, off, D * F, Ly.w_2);
    }
    off = load_tensor(*d, img, off, D, M->g_out);
    off = load_tensor(*d, img, off, V * D, M->w_head);
    if (off != bytes) {
        std::fprintf(stderr, "orc_model_create: weight image is %zu bytes, expected %zu\n", bytes, off);
        delete M;
        return nullptr;
    }
    return M;
}

void orc_model_destroy(void* m) { delete (Model*)m; }

// seq: [len] with seq[0] ignored (class token), logits: [len][V]
void orc_forward_full(void* m, int label, const int32_t* seq, int len, float* logits) {
    forward_full(*(Model*)m, label, seq, len, logits);
}

// Windowed forward over an external cache kc/vc [L][T][D] (fp32).  logits may be null.
void orc_forward_window(void* m, float* kc, float* vc, int label, const int32_t* seq, int c, int n, float* logits) {
    forward_window(*(Model*)m, kc, vc, label, seq, c, n, logits);
}

// As orc_forward_window, also copying the intermediates of layer tr->layer (component parity tests).
void orc_forward_window_trace(void* m, float* kc, float* vc, int label, const int32_t* seq, int c, int n,
                              float* logits, const Trace* tr) {
    forward_window(*(Model*)m, kc, vc, label, seq, c, n, logits, tr);
}

// Single stages of one decoder block on caller-supplied inputs (component parity tests feed them the GPU's own
// intermediates, so that each kernel is compared on identical inputs).  Same functions as forward_window runs.
void orc_stage_qkv(void* m, int layer, const float* x, int n, int c, float* a, float* qkv) {
    const Model& M = *(Model*)m;
    stage_qkv(M, M.layers[layer], x, n, c, a, qkv);
}
void orc_stage_attend(void* m, const float* q, const float* K, const float* V, int c, int n, float* o) {
    const Model& M = *(Model*)m;
    stage_attend(M, q, (size_t)M.d.D, K, V, c, n, o);
}
void orc_stage_attn_out(void* m, int layer, const float* o, int n, float* x) {
    const Model& M = *(Model*)m;
    stage_attn_out(M, M.layers[layer], o, n, x);
}
void orc_stage_ffn_act(void* m, int layer, const float* x, int n, float* mm, float* act) {
    const Model& M = *(Model*)m;
    stage_ffn_act(M, M.layers[layer], x, n, mm, act);
}
void orc_stage_ffn_down(void* m, int layer, const float* act, int n, float* x) {
    const Model& M = *(Model*)m;
    stage_ffn_down(M, M.layers[layer], act, n, x);
}

// Diagnostics for the noise-floor calibration (both 0: the oracle proper).  Never a comparison target.
void orc_model_set_diag(void* m, int acc_f32, int attn_w_bf16, int norm_folded) {
    ((Model*)m)->acc_f32 = acc_f32;
    ((Model*)m)->attn_w_bf16 = attn_w_bf16;
    ((Model*)m)->norm_folded = norm_folded;
}

void orc_probs(const float* lc, const float* lu, float s, float tau, int k, int V, float* p) {
    probs(lc, lu, s, tau, k, V, p);
}

int orc_sample(const float* a, int V, uint32_t word) { return sample_fixed(a, V, word); }

// One image's verification / commit / refresh on caller-supplied probabilities
// and random words (used for brute-force pins and for replaying a GPU round).
int orc_decide(int V, int T, int W, int H, int greedy, int32_t* c_inout, int32_t* seq, uint8_t* delta,
               const float* p, int n, const float* qprev, int qbase, const uint32_t* words, const uint32_t* w3_beyond,
               int32_t* j_out) {
    int c = *c_inout, j = -1;
    const int m = decide_and_refresh(V, T, W, H, greedy != 0, c, seq, delta, p, n, qprev, qbase,
                                     (const uint32_t (*)[4])words, w3_beyond, &j);
    *c_inout = c;
    *j_out = j;
    return m;
}

// As orc_decide, with the words drawn from Philox keyed (seed; image id, position, round).
// m_limit > 0: batch-synchronous truncation as in decide_and_refresh.
int orc_replay_round(int V, int T, int W, int H, int greedy, uint64_t seed, int id, uint32_t round,
                     int32_t* c_inout, int32_t* seq, uint8_t* delta, const float* p, const float* qprev, int qbase,
                     int32_t* j_out, int m_limit) {
    Params P{};
    P.seed = seed;
    int c = *c_inout, j = -1;
    const int n = std::min(W, T - c);
    std::vector<uint32_t> words((size_t)n * 4), beyond(W);
    for (int i = 0; i < n; ++i) words_for(P, id, c + i + 1, round, &words[(size_t)i * 4]);
    for (int d = 0; d < W; ++d) {
        uint32_t w[4];
        words_for(P, id, c + n + 1 + d, round, w);
        beyond[d] = w[3];
    }
    const int m = decide_and_refresh(V, T, W, H, greedy != 0, c, seq, delta, p, n, qprev, qbase,
                                     (const uint32_t (*)[4])words.data(), beyond.data(), &j, m_limit);
    *c_inout = c;
    *j_out = j;
    return m;
}

// Rollout state: init + prefill + initial windows.  image_ids (may be null)
// gives each image's index for the random-number key (default: 0..B-1).
void* orc_rollout_create(void* m, int B, const int32_t* prefix_tokens, const int32_t* prefix_len,
                         const int32_t* labels, const int32_t* image_ids, const Params* P) {
    const Model& M = *(Model*)m;
    Rollout* R = new Rollout();
    R->M = &M;
    R->P = *P;
    R->B = B;
    R->round = 0;
    R->img.resize(B);
    const int T = M.T, V = M.d.V, W = P->window;
    const bool cfg = P->cfg_scale != 1.0f;
    const size_t cache = (size_t)M.d.L * T * M.d.D;
    // one image per thread when there are enough images; otherwise the matrix products use the threads
#pragma omp parallel for schedule(dynamic) if (B >= omp_get_max_threads())
    for (int b = 0; b < B; ++b) {
        Image& im = R->img[b];
        im.id = image_ids ? image_ids[b] : b;
        im.label = labels[b];
        im.k = prefix_len[b];
        im.c = im.k;
        im.qbase = 0;
        im.seq.assign(T + 1, 0);
        im.delta.assign(T + 1, 0);
        for (int t = 1; t <= im.k; ++t) im.seq[t] = prefix_tokens[(size_t)b * T + (t - 1)];
        im.kc.assign(cache, 0.f);
        im.vc.assign(cache, 0.f);
        if (cfg) {
            im.ku.assign(cache, 0.f);
            im.vu.assign(cache, 0.f);
        }
        im.pcur.assign((size_t)W * V, 0.f);
        im.pprev.assign((size_t)W * V, 0.f);
        im.logc.assign((size_t)W * V, 0.f);
        if (cfg) im.logu.assign((size_t)W * V, 0.f);
        prefill(*R, im);
        init_window(*R, im);
    }
    return R;
}

void orc_rollout_destroy(void* r) { delete (Rollout*)r; }

int orc_rollout_live(void* r) {
    Rollout* R = (Rollout*)r;
    int a = 0;
    for (auto& im : R->img) a += im.c < R->M->T;
    return a;
}

// One round over every live image.  m_out[B] (may be null) receives the tokens
// committed per image (0 for finished images); j_out[B] the first-reject index
// (-1 none / not run).  Returns the live count AFTER the round.
int orc_rollout_round(void* r, int32_t* m_out, int32_t* j_out) {
    Rollout* R = (Rollout*)r;
    const int T = R->M->T;
    int live = 0;
    for (auto& im : R->img) live += im.c < T;
    if (live == 0) return 0;
    // Eq. 6: Full iff A > gamma (mode affects which rows run, never the values)
    const bool sync = R->P.exec_mode == 3;
    int mode = R->P.exec_mode == 2 ? (live > R->P.gamma ? 0 : 1) : (sync ? 0 : R->P.exec_mode);
    R->trace_live.push_back(live);
    R->trace_mode.push_back(mode);
    long long commits = 0, rej = 0;
    int m_limit = 0;
    if (sync) {
        // batch-synchronous progress: every live image advances by the smallest commit of the batch
        std::vector<int> nat(R->B, 0);
#pragma omp parallel for schedule(dynamic) if (live >= omp_get_max_threads())
        for (int b = 0; b < R->B; ++b) {
            Image& im = R->img[b];
            if (im.c < T) {
                image_forward(*R, im);
                nat[b] = image_natural_commit(*R, im);
            }
        }
        for (int b = 0; b < R->B; ++b)
            if (R->img[b].c < T && (m_limit == 0 || nat[b] < m_limit)) m_limit = nat[b];
    }
#pragma omp parallel for schedule(dynamic) reduction(+ : commits, rej) if (live >= omp_get_max_threads())
    for (int b = 0; b < R->B; ++b) {
        Image& im = R->img[b];
        int m = 0, j = -1;
        if (im.c < T) {
            m = sync ? image_commit(*R, im, &j, m_limit) : image_round(*R, im, &j);
            commits += m;
            rej += (j >= 0);
        }
        if (m_out) m_out[b] = m;
        if (j_out) j_out[b] = j;
    }
    R->image_forwards += live;
    R->committed += commits;
    R->rejects += rej;
    R->round += 1;
    int after = 0;
    for (auto& im : R->img) after += im.c < T;
    return after;
}

int orc_rollout_run(void* r, int max_rounds) {
    int n = 0;
    while (orc_rollout_live(r) > 0 && (max_rounds <= 0 || n < max_rounds)) {
        orc_rollout_round(r, nullptr, nullptr);
        ++n;
    }
    return n;
}

void orc_rollout_tokens(void* r, int32_t* out /*[B][T]*/) {
    Rollout* R = (Rollout*)r;
    const int T = R->M->T;
    for (int b = 0; b < R->B; ++b)
        for (int t = 1; t <= T; ++t) out[(size_t)b * T + t - 1] = R->img[b].seq[t];
}

// state export: cursor[B], seq[B][T+1], delta[B][T+1], qbase[B]; returns the round counter
int orc_rollout_get_state(void* r, int32_t* cursor, int32_t* seq, uint8_t* delta, int32_t* qbase) {
    Rollout* R = (Rollout*)r;
    const int T = R->M->T;
    for (int b = 0; b < R->B; ++b) {
        const Image& im = R->img[b];
        cursor[b] = im.c;
        qbase[b] = im.qbase;
        std::memcpy(seq + (size_t)b * (T + 1), im.seq.data(), (T + 1) * 4);
        std::memcpy(delta + (size_t)b * (T + 1), im.delta.data(), T + 1);
    }
    return R->round;
}

// Last round's probabilities of image b: rows 0..n-1 of [W][V] (these are the
// next round's proposals).  Returns n.
int orc_rollout_probs(void* r, int b, float* out) {
    Rollout* R = (Rollout*)r;
    const Image& im = R->img[b];
    std::memcpy(out, im.pprev.data(), (size_t)im.last_n * R->M->d.V * 4);
    return im.last_n;
}

// Last round's logits of image b, branch 0 = conditional, 1 = unconditional.  Returns n.
int orc_rollout_logits(void* r, int b, int branch, float* out) {
    Rollout* R = (Rollout*)r;
    const Image& im = R->img[b];
    const std::vector<float>& src = branch ? im.logu : im.logc;
    if (src.empty()) return 0;
    std::memcpy(out, src.data(), (size_t)im.last_n * R->M->d.V * 4);
    return im.last_n;
}

// stats: rounds, image_forwards, committed, rejects; traces of length rounds
int orc_rollout_stats(void* r, int64_t* out4, int32_t* live_trace, int32_t* mode_trace, int cap) {
    Rollout* R = (Rollout*)r;
    out4[0] = (int64_t)R->trace_live.size();
    out4[1] = R->image_forwards;
    out4[2] = R->committed;
    out4[3] = R->rejects;
    const int n = std::min<int>(cap, (int)R->trace_live.size());
    for (int i = 0; i < n; ++i) {
        if (live_trace) live_trace[i] = R->trace_live[i];
        if (mode_trace) mode_trace[i] = R->trace_mode[i];
    }
    return (int)R->trace_live.size();
}

// Plain autoregressive sampler (Eq. 1 / Eq. 2): for t = k+1..T recompute the
// whole sequence without a cache and sample x_t with word 1 of
// (image, t, round = t-k-1).  greedy: argmax instead.
void orc_ar_rollout(void* m, int B, const int32_t* prefix_tokens, const int32_t* prefix_len, const int32_t* labels,
                    const int32_t* image_ids, const Params* P, int32_t* out /*[B][T]*/) {
    const Model& M = *(Model*)m;
    const int T = M.T, V = M.d.V;
    const bool cfg = P->cfg_scale != 1.0f;
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        std::vector<int32_t> seq(T + 1, 0);
        const int k = prefix_len[b];
        const int id = image_ids ? image_ids[b] : b;
        for (int t = 1; t <= k; ++t) seq[t] = prefix_tokens[(size_t)b * T + t - 1];
        std::vector<float> lc((size_t)T * V), lu, p(V);
        if (cfg) lu.resize((size_t)T * V);
        for (int t = k + 1; t <= T; ++t) {
            forward_full(M, labels[b], seq.data(), t, lc.data());
            if (cfg) forward_full(M, M.d.C, seq.data(), t, lu.data());
            probs(&lc[(size_t)(t - 1) * V], cfg ? &lu[(size_t)(t - 1) * V] : nullptr, P->cfg_scale, P->temperature,
                  P->top_k, V, p.data());
            if (P->verify_mode == 1) {
                seq[t] = argmax_low(p.data(), V);
            } else {
                uint32_t w[4];
                words_for(*P, id, t, (uint32_t)(t - k - 1), w);
                seq[t] = sample_fixed(p.data(), V, w[1]);
            }
        }
        for (int t = 1; t <= T; ++t) out[(size_t)b * T + t - 1] = seq[t];
    }
}

// ------------------------------------------------------- distillation score (Eq. 3)

// D_biKL(p, q) = 1/2 KL(p || q) + 1/2 KL(q || p) for p = softmax(s), q = softmax(t),
// the definition written out in the log domain, double throughout.
double bikl_row(const float* s, const float* t, int V) {
    double ms = s[0], mt = t[0];
    for (int v = 1; v < V; ++v) {
        if (s[v] > ms) ms = s[v];
        if (t[v] > mt) mt = t[v];
    }
    double zs = 0.0, zt = 0.0;
    for (int v = 0; v < V; ++v) {
        zs += std::exp((double)s[v] - ms);
        zt += std::exp((double)t[v] - mt);
    }
    const double lzs = std::log(zs), lzt = std::log(zt);
    double kl_pq = 0.0, kl_qp = 0.0;
    for (int v = 0; v < V; ++v) {
        const double lp = (double)s[v] - ms - lzs, lq = (double)t[v] - mt - lzt;
        kl_pq += std::exp(lp) * (lp - lq);
        kl_qp += std::exp(lq) * (lq - lp);
    }
    return 0.5 * kl_pq + 0.5 * kl_qp;
}

void orc_bikl(const float* s, const float* t, int rows, int V, double* out) {
    for (int r = 0; r < rows; ++r) out[r] = bikl_row(s + (size_t)r * V, t + (size_t)r * V, V);
}

// Eq. 3 on completed trajectories: for image b with real prefix k_b, the mean over t = k_b+1..T of
// D_biKL(p_S(. | x_<t), p_T(. | x_<t)); both models see the same tokens and the image's class, no
// guidance, no temperature, no top-k.  pos [B][T]: entry t-1 holds the term of position t (0 for t <= k_b);
// per_image [B] (0 when k_b = T); *loss = mean of per_image over the images with k_b < T.
void orc_score(void* student, void* teacher, int B, const int32_t* tokens, const int32_t* prefix_len,
               const int32_t* labels, double* pos, double* per_image, double* loss) {
    const Model& S = *(Model*)student;
    const Model& Tm = *(Model*)teacher;
    const int T = S.T, V = S.d.V;
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        std::vector<int32_t> seq(T + 1, 0);
        for (int t = 1; t <= T; ++t) seq[t] = tokens[(size_t)b * T + t - 1];
        std::vector<float> ls((size_t)T * V), lt((size_t)T * V);
        // inputs are sequence indices 0..T-1 (class token, x_1..x_{T-1}); output row i is the distribution of x_{i+1}
        forward_full(S, labels[b], seq.data(), T, ls.data());
        forward_full(Tm, labels[b], seq.data(), T, lt.data());
        const int k = prefix_len[b];
        double sum = 0.0;
        for (int t = 1; t <= T; ++t) {
            double d = 0.0;
            if (t >= k + 1) d = bikl_row(&ls[(size_t)(t - 1) * V], &lt[(size_t)(t - 1) * V], V);
            pos[(size_t)b * T + t - 1] = d;
            sum += d;
        }
        per_image[b] = k < T ? sum / (double)(T - k) : 0.0;
    }
    double tot = 0.0;
    int cnt = 0;
    for (int b = 0; b < B; ++b)
        if (prefix_len[b] < T) {
            tot += per_image[b];
            ++cnt;
        }
    *loss = cnt ? tot / cnt : 0.0;
}

int orc_num_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
