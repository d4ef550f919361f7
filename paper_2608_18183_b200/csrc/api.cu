// C ABI of the rollout library (see include/hbsjd.h): context, host-side round loop, debug helpers.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <type_traits>
#include <vector>

#include "../../include/hbsjd.h"
#include "internal.h"

using namespace hbsjd;

namespace {

constexpr int PAGE_TOKENS = 64;

struct LayerW {
    const void *g_attn, *w_qkv, *w_o, *g_ffn, *w_13, *w_2;
};

}  // namespace

struct hbsjd_ctx {
    hbsjd_model_desc d;
    int T, dh, Bmax, Wmax;
    bool bf16_model;
    bool fold_norm;      // bf16 model: RMSNorm folded into the GEMM epilogues (launch-bound contexts), else its own kernel
    bool unit_gains;     // every norm gain of the model is exactly 1
    bool ref_attention;  // debugging: run the one-warp-per-row attention kernel
    cudaStream_t stream;
    // weights
    unsigned char* w_img;
    const void *tok_emb, *cls_emb, *g_out, *w_head;
    std::vector<LayerW> layers;
    float* rope_cs;
    // KV pages
    void *kc, *vc;
    int32_t* page_table;
    int pages_per_row, n_pages;
    // rollout state
    State st;
    float* pbuf[2];
    int parity;
    uint8_t* flag;
    int32_t *cand_rep, *cand_ref;
    // activations
    float *h, *qkv, *gu, *logits;
    void *a, *q, *o, *act;  // a: normed operand (fp32 model) / bf16 copy of the residual stream (bf16 model)
    float* ssq;             // [rows][dim / 32] partial sums of squares of the residual rows (bf16 model)
    // host side
    int32_t* h_counters;  // pinned [8]
    cudaEvent_t ev0, ev1, ev2;
    hbsjd_params P;
    bool have_rollout;
    int live, round, last_S, last_compact;
    int dbg_layer;  // layer of the last hbsjd_debug_forward (-1: none); selects the KV rows of hbsjd_debug_read
    hbsjd_stats stats;
    long long launches;
    // host-buffer staging
    int32_t *stage_tok, *stage_len, *stage_lab, *stage_out;
    void* verify_scratch;
    float *score_pos, *score_img, *score_loss;  // [Bmax][T], [Bmax], [1]
    int32_t* m_sync;                              // [1] smallest commit of the round (batch-synchronous progress)
    // per-class event timing
    bool profiling;
    struct ProfSlot { cudaEvent_t a, b; int cls; double work; int rows; double bytes; };
    std::vector<ProfSlot> pool;
    int pool_used;
    int pending_attn;  // attention launches of the current forward whose byte count waits for the counters
    hbsjd_kernel_profile prof;
    char err[256];
};

namespace {

#define CK(call)                                                                                  \
    do {                                                                                          \
        cudaError_t e_ = (call);                                                                  \
        if (e_ != cudaSuccess) {                                                                  \
            snprintf(c->err, sizeof(c->err), "%s: %s", #call, cudaGetErrorString(e_));            \
            return e_ == cudaErrorMemoryAllocation ? HBSJD_ENOMEM : HBSJD_ECUDA;                  \
        }                                                                                         \
    } while (0)

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// Brackets the launches issued between prof_begin and prof_end with an event pair of class `cls`.
int prof_begin(hbsjd_ctx* c, int cls, double work, int rows = 0, double bytes = 0.0) {
    if (!c->profiling) return -1;
    if (c->pool_used >= (int)c->pool.size()) {
        c->prof.dropped++;
        return -1;
    }
    hbsjd_ctx::ProfSlot& s = c->pool[c->pool_used];
    s.cls = cls;
    s.work = work;
    s.rows = rows;
    s.bytes = bytes;
    cudaEventRecord(s.a, c->stream);
    return c->pool_used++;
}
void prof_end(hbsjd_ctx* c, int slot) {
    if (slot >= 0) cudaEventRecord(c->pool[slot].b, c->stream);
}
// After a stream synchronisation: folds the finished event pairs into the totals.  attn_bytes is the
// algorithmic traffic of each attention launch of the forward just finished.
void prof_resolve(hbsjd_ctx* c, double attn_bytes, double accept_bytes) {
    for (int i = 0; i < c->pool_used; ++i) {
        hbsjd_ctx::ProfSlot& s = c->pool[i];
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, s.a, s.b) != cudaSuccess) continue;
        double work = s.work;
        if (s.cls == HBSJD_PROF_ATTENTION) work = attn_bytes;
        if (s.cls == HBSJD_PROF_ACCEPT) work = accept_bytes;
        c->prof.ms[s.cls] += ms;
        c->prof.work[s.cls] += work;
        c->prof.launches[s.cls] += 1;
        if (s.cls == HBSJD_PROF_GEMM && s.rows > 0) {
            const int bin = s.rows <= 512 ? 0 : s.rows <= 2048 ? 1 : s.rows <= 6144 ? 2 : 3;
            c->prof.gemm_ms_by_rows[bin] += ms;
            c->prof.gemm_work_by_rows[bin] += work;
            c->prof.gemm_bytes_by_rows[bin] += s.bytes;
            c->prof.gemm_launches_by_rows[bin] += 1;
        }
    }
    c->pool_used = 0;
}

template <typename T>
int dev_alloc(hbsjd_ctx* c, T** p, size_t count) {
    *p = nullptr;
    CK(cudaMalloc((void**)p, count * sizeof(T) > 0 ? count * sizeof(T) : 16));
    CK(cudaMemsetAsync(*p, 0, count * sizeof(T), c->stream));
    return 0;
}

KvView kv_view(const hbsjd_ctx* c) {
    KvView kv;
    kv.k = c->kc;
    kv.v = c->vc;
    kv.table = c->page_table;
    kv.pages_per_row = c->pages_per_row;
    kv.page = PAGE_TOKENS;
    kv.n_pages = c->n_pages;
    kv.D = c->d.dim;
    return kv;
}

// m_cap: row capacity of the A and C buffers when they are the context's own (0: exactly M rows)
// w_constant: W is one of the model's weight matrices (see gemm_tcgen05_run)
template <typename TA>
int gemm(hbsjd_ctx* c, const void* A, const void* W, float* C, int M, int N, int K, int accumulate, int m_cap = 0,
         int w_constant = 1, unsigned int acc_wait_ns = 0, int tile = 0);

template <>
int gemm<float>(hbsjd_ctx* c, const void* A, const void* W, float* C, int M, int N, int K, int accumulate, int, int,
                unsigned int, int) {
    const int ps = prof_begin(c, HBSJD_PROF_GEMM, 2.0 * M * N * K, M,
                              4.0 * ((double)M * K + (double)N * K) + 4.0 * M * N * (accumulate ? 2 : 1));
    launch_gemm_simt<float>((const float*)A, (const float*)W, C, M, N, K, accumulate, c->stream);
    prof_end(c, ps);
    c->launches++;
    return 0;
}

template <>
int gemm<bf16>(hbsjd_ctx* c, const void* A, const void* W, float* C, int M, int N, int K, int accumulate,
               int m_cap, int w_constant, unsigned int acc_wait_ns, int tile) {
    c->launches++;
    const int ps = prof_begin(c, HBSJD_PROF_GEMM, 2.0 * M * N * K, M,
                              2.0 * ((double)M * K + (double)N * K) + 4.0 * M * N * (accumulate ? 2 : 1));
    const int rc = gemm_tcgen05_run((const bf16*)A, (const bf16*)W, C, M, N, K, accumulate, tile, m_cap,
                                    c->st.counters + CNT_ERROR, c->stream, c->err, sizeof(c->err), w_constant,
                                    acc_wait_ns);
    prof_end(c, ps);
    return rc == 0 ? 0 : (rc == -1 ? HBSJD_EINVAL : HBSJD_ECUDA);
}

// One batched verifier forward over S slots (Sec. 4.2 "Batched verification").
// stop_layer >= 0 (debugging): return after the attention sub-block (stop_stage 0) or the whole block
// (stop_stage 1) of that layer, leaving the activation buffers as that point found them.
template <typename TA>
int forward(hbsjd_ctx* c, int S, bool want_logits, int stop_layer = -1, int stop_stage = 0);

// fp32 model: every step its own kernel (the configuration exists for parity, not speed).
template <>
int forward<float>(hbsjd_ctx* c, int S, bool want_logits, int stop_layer, int stop_stage) {
    typedef float TA;
    const State& st = c->st;
    const int M = st.nb * S * st.W, D = st.D, F = st.F;
    cudaStream_t s = c->stream;
    const KvView kv = kv_view(c);
    launch_embed<TA>(st, S, (const TA*)c->tok_emb, (const TA*)c->cls_emb, c->h, nullptr, nullptr, s);
    c->launches++;
    auto norm = [&](const float* x, const void* gain) {
        const int ps = prof_begin(c, HBSJD_PROF_OTHER, (double)M * D * (4.0 + sizeof(TA)));
        launch_rmsnorm<TA>(x, (const TA*)gain, (TA*)c->a, M, D, c->d.rms_eps, s);
        prof_end(c, ps);
        c->launches++;
    };
    for (int l = 0; l < st.L; ++l) {
        const LayerW& w = c->layers[l];
        int rc;
        norm(c->h, w.g_attn);
        if ((rc = gemm<TA>(c, c->a, w.w_qkv, c->qkv, M, 3 * D, D, 0))) return rc;
        launch_rope_kv<TA>(st, S, l, c->qkv, c->rope_cs, (TA*)c->q, kv, s);
        c->launches++;
        {
            const int ps = prof_begin(c, HBSJD_PROF_ATTENTION, 0.0);
            launch_attention_ref<TA>(st, S, l, (const TA*)c->q, kv, (TA*)c->o, s);
            prof_end(c, ps);
            c->launches++;
        }
        if ((rc = gemm<TA>(c, c->o, w.w_o, c->h, M, D, D, 1))) return rc;
        if (l == stop_layer && stop_stage == 0) return 0;
        norm(c->h, w.g_ffn);
        if ((rc = gemm<TA>(c, c->a, w.w_13, c->gu, M, 2 * F, D, 0))) return rc;
        launch_swiglu<TA>(c->gu, (TA*)c->act, M, F, s);
        c->launches++;
        if ((rc = gemm<TA>(c, c->act, w.w_2, c->h, M, D, F, 1))) return rc;
        if (l == stop_layer) return 0;
    }
    if (want_logits) {
        norm(c->h, c->g_out);
        int rc;
        if ((rc = gemm<TA>(c, c->a, c->w_head, c->logits, M, st.V, D, 0))) return rc;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(c->err, sizeof(c->err), "forward launch: %s", cudaGetErrorString(e));
        return HBSJD_ECUDA;
    }
    return 0;
}

// bf16 model: four tensor-core GEMMs and one attention kernel per layer; RoPE + the paged KV write, SwiGLU and the
// residual add ride in the GEMM epilogues.  RMSNorm comes in two forms, fixed per context at creation:
//   folded (contexts of at most 2048 activation rows, which are bound by the number of launches): no kernel of its
//     own -- the kernels that write the residual stream (embedding gather, attention-out and FFN-down projections)
//     also leave its bf16 copy and per-row partial sums of squares, the norm's gain is folded into the following
//     weight matrix at load, and the following GEMM's epilogue applies the row factor rsqrt(mean(x^2) + eps);
//   separate (larger contexts): one warp-per-row kernel in front of the QKV, gate/up and head projections, and the
//     residual update as a bulk tensor reduce-add from the epilogue.  At 8192 rows the folded residual update costs
//     what the separate kernel costs (its reads of the old residual compete with the operand stream for L2
//     bandwidth), so the form with the exact operand rounding of the definition is kept there.
template <>
int forward<bf16>(hbsjd_ctx* c, int S, bool want_logits, int stop_layer, int stop_stage) {
    const State& st = c->st;
    const int M = st.nb * S * st.W, D = st.D, F = st.F;
    const int Mcap = 2 * c->Bmax * c->Wmax;  // row capacity of the activation buffers
    cudaStream_t s = c->stream;
    const KvView kv = kv_view(c);
    const bool fold = c->fold_norm;
    const double es = 2.0;  // bytes of a bf16 operand / output element (algorithmic byte counts of the profile)
    bf16* a = (bf16*)c->a;  // folded: bf16 copy of the residual stream; separate: the normed operand
    const NormIn nin = {fold ? c->ssq : nullptr, c->d.rms_eps};
    int32_t* eflag = c->st.counters + CNT_ERROR;
    auto done = [&](int rc) { return rc == 0 ? 0 : (rc == -1 ? HBSJD_EINVAL : HBSJD_ECUDA); };
    auto norm = [&](const void* gain) {  // separate form only
        const int ps = prof_begin(c, HBSJD_PROF_OTHER, (double)M * D * (4.0 + 2.0));
        launch_rmsnorm<bf16>(c->h, (const bf16*)gain, a, M, D, c->d.rms_eps, s);
        prof_end(c, ps);
        c->launches++;
    };
    // residual update h += A W^T
    auto residual = [&](const void* A, const void* W, int K) {
        // operands, the fp32 residual read and written, and (folded norm) its bf16 copy
        const int ps = prof_begin(c, HBSJD_PROF_GEMM, 2.0 * M * D * K, M,
                                  es * ((double)M * K + (double)D * K) + 8.0 * M * D + (fold ? 2.0 * M * D : 0.0));
        int rc;
        if (fold)
            rc = gemm_tcgen05_addnorm((const bf16*)A, (const bf16*)W, c->h, a, c->ssq, M, D, K, Mcap, eflag, s, c->err,
                                      sizeof(c->err));
        else
            rc = gemm_tcgen05_run((const bf16*)A, (const bf16*)W, c->h, M, D, K, 1, 0, Mcap, eflag, s, c->err,
                                  sizeof(c->err));
        prof_end(c, ps);
        c->launches++;
        return rc;
    };
    launch_embed<bf16>(st, S, (const bf16*)c->tok_emb, (const bf16*)c->cls_emb, c->h, fold ? a : nullptr,
                       fold ? c->ssq : nullptr, s);
    c->launches++;
    for (int l = 0; l < st.L; ++l) {
        const LayerW& w = c->layers[l];
        int rc, ps;
        if (!fold) norm(w.g_attn);
        ps = prof_begin(c, HBSJD_PROF_GEMM, 2.0 * M * 3 * D * D, M,
                        es * ((double)M * D + 3.0 * D * D) + es * 3.0 * M * D);  // q, k, v written
        rc = gemm_tcgen05_qkv(a, (const bf16*)w.w_qkv, (bf16*)c->q, st, S, l, c->rope_cs, kv, Mcap, nin, eflag, s,
                              c->err, sizeof(c->err));
        prof_end(c, ps);
        if (rc) return done(rc);
        ps = prof_begin(c, HBSJD_PROF_ATTENTION, 0.0);
        if (attention_tma_supported(st, kv)) {
            rc = launch_attention_tma(st, S, l, (const bf16*)c->q, Mcap, kv, (bf16*)c->o, eflag, s, c->err,
                                      sizeof(c->err));
            if (rc) return HBSJD_ECUDA;
        } else {
            launch_attention_ref<bf16>(st, S, l, (const bf16*)c->q, kv, (bf16*)c->o, s);
        }
        prof_end(c, ps);
        c->launches += 2;
        if ((rc = residual(c->o, w.w_o, D))) return done(rc);
        if (l == stop_layer && stop_stage == 0) return 0;
        if (!fold) norm(w.g_ffn);
        ps = prof_begin(c, HBSJD_PROF_GEMM, 2.0 * M * 2 * F * D, M,
                        es * ((double)M * D + 2.0 * F * D) + es * (double)M * F);
        rc = gemm_tcgen05_swiglu(a, (const bf16*)w.w_13, (bf16*)c->act, M, 2 * F, D, Mcap, nin, eflag, s, c->err,
                                 sizeof(c->err));
        prof_end(c, ps);
        if (rc) return done(rc);
        c->launches++;
        if ((rc = residual(c->act, w.w_2, F))) return done(rc);
        if (l == stop_layer) return 0;
    }
    if (want_logits) {
        if (!fold) norm(c->g_out);
        const int ps = prof_begin(c, HBSJD_PROF_GEMM, 2.0 * M * st.V * D, M,
                                  es * ((double)M * D + (double)st.V * D) + 4.0 * M * st.V);
        const int rc = gemm_tcgen05_head(a, (const bf16*)c->w_head, c->logits, M, st.V, D, Mcap, nin, eflag, s,
                                         c->err, sizeof(c->err));
        prof_end(c, ps);
        if (rc) return done(rc);
        c->launches++;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(c->err, sizeof(c->err), "forward launch: %s", cudaGetErrorString(e));
        return HBSJD_ECUDA;
    }
    return 0;
}

int forward_any(hbsjd_ctx* c, int S, bool want_logits, int stop_layer = -1, int stop_stage = 0) {
    return c->bf16_model ? forward<bf16>(c, S, want_logits, stop_layer, stop_stage)
                         : forward<float>(c, S, want_logits, stop_layer, stop_stage);
}

int choose_compact(const hbsjd_ctx* c, int live) {
    if (c->P.exec_mode == HBSJD_EXEC_FULL || c->P.exec_mode == HBSJD_EXEC_SYNC) return 0;
    if (c->P.exec_mode == HBSJD_EXEC_COMPACT) return 1;
    return live > c->P.gamma ? 0 : 1;  // Eq. 6
}

int sync_counters(hbsjd_ctx* c) {
    CK(cudaMemcpyAsync(c->h_counters, c->st.counters, 8 * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (c->profiling) {
        // algorithmic bytes of the forward just finished, from the slot set-up sums:
        // attention per layer: K and V rows 0..c+n-1 read per row, q read and output written per input;
        // accept: logits of every branch read, probabilities written, per input
        const double es = c->bf16_model ? 2.0 : 4.0, D = c->d.dim, V = c->d.vocab, nb = c->st.nb;
        const double keys = c->h_counters[CNT_SUM_KEYS], n = c->h_counters[CNT_SUM_N];
        prof_resolve(c, nb * (keys * 2.0 * D * es + n * 2.0 * D * es), n * (nb + 1.0) * V * 4.0);
    }
    if (c->h_counters[CNT_ERROR] != 0) {
        const int code = c->h_counters[CNT_ERROR];
        cudaMemsetAsync(c->st.counters + CNT_ERROR, 0, sizeof(int32_t), c->stream);
        if (code >= 16) {  // a kernel met rollout state that cannot be valid; it skipped the access
            snprintf(c->err, sizeof(c->err), "invalid rollout state on the device (code %d: %s)", code,
                     code == 16 ? "cursor out of range" : code == 17 ? "draft token out of range"
                                                                     : "proposal row out of range");
            return HBSJD_EINVAL;
        }
        snprintf(c->err, sizeof(c->err), "a bounded device-side wait gave up (code %d)", code);
        return HBSJD_ETIMEOUT;
    }
    return 0;
}

int run_round(hbsjd_ctx* c) {
    if (c->live == 0) return 0;
    const int compact = choose_compact(c, c->live);
    const int S = compact ? c->live : c->st.B;
    launch_setup(c->st, 0, compact, c->stream);
    c->launches++;
    int rc = forward_any(c, S, true);
    if (rc) return rc;
    AcceptArgs a;
    a.logits = c->logits;
    a.pcur = c->pbuf[c->parity];
    a.pprev = c->pbuf[c->parity ^ 1];
    a.flag = c->flag;
    a.cand_rep = c->cand_rep;
    a.cand_ref = c->cand_ref;
    a.S = S;
    a.cfg_scale = c->P.cfg_scale;
    a.temperature = c->P.temperature;
    a.top_k = c->P.top_k;
    a.greedy = c->P.verify_mode == HBSJD_VERIFY_GREEDY;
    a.seed_lo = (uint32_t)(c->P.seed & 0xffffffffu);
    a.seed_hi = (uint32_t)(c->P.seed >> 32);
    a.round = (uint32_t)c->round;
    a.m_sync = c->P.exec_mode == HBSJD_EXEC_SYNC ? c->m_sync : nullptr;
    {
        const int ps = prof_begin(c, HBSJD_PROF_ACCEPT, 0.0);
        launch_prob_accept(c->st, a, c->stream);
        if (a.m_sync) {
            launch_sync_min(c->st, a, c->m_sync, c->stream);
            c->launches++;
        }
        launch_commit(c->st, a, c->stream);
        prof_end(c, ps);
    }
    c->launches += 2;
    CK(cudaGetLastError());
    rc = sync_counters(c);
    if (rc) return rc;
    if (c->h_counters[CNT_LIVE_SETUP] != c->live) {
        snprintf(c->err, sizeof(c->err), "live count mismatch: host %d device %d", c->live,
                 c->h_counters[CNT_LIVE_SETUP]);
        return HBSJD_ESTATE;
    }
    c->stats.rounds += 1;
    c->stats.image_forwards += c->live;
    if (compact) c->stats.compact_rounds += 1;
    else c->stats.full_rounds += 1;
    c->stats.committed = c->h_counters[CNT_COMMITTED];
    c->stats.rejects = c->h_counters[CNT_REJECTS];
    c->live = c->h_counters[CNT_LIVE];
    c->last_S = S;
    c->last_compact = compact;
    c->round += 1;
    c->parity ^= 1;
    return 0;
}

void free_all(hbsjd_ctx* c) {
    void* ptrs[] = {c->w_img, c->rope_cs, c->kc, c->vc, c->page_table, c->st.cursor, c->st.seq, c->st.delta,
                    c->st.qbase, c->st.label, c->st.klen, c->st.pfill, c->st.slot_img, c->st.slot_c, c->st.slot_n, c->st.slot_order,
                    c->st.counters, c->st.m_last, c->st.j_last, c->pbuf[0], c->pbuf[1], c->flag, c->cand_rep,
                    c->cand_ref, c->h, c->qkv, c->gu, c->logits, c->a, c->q, c->o, c->act, c->ssq,
                    c->stage_tok, c->stage_len, c->stage_lab, c->stage_out, c->verify_scratch,
                    c->score_pos, c->score_img, c->score_loss, c->m_sync};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    if (c->h_counters) cudaFreeHost(c->h_counters);
    for (auto& s : c->pool) {
        if (s.a) cudaEventDestroy(s.a);
        if (s.b) cudaEventDestroy(s.b);
    }
    if (c->ev0) cudaEventDestroy(c->ev0);
    if (c->ev1) cudaEventDestroy(c->ev1);
    if (c->ev2) cudaEventDestroy(c->ev2);
}

int create_impl(hbsjd_ctx* c, const void* weights, size_t weight_bytes) {
    const hbsjd_model_desc& d = c->d;
    const size_t D = d.dim, F = d.ffn_hidden, V = d.vocab, L = d.n_layers;
    const size_t es = c->bf16_model ? 2 : 4;
    // weight image offsets (each tensor on a 256-byte boundary)
    size_t off = 0;
    auto take = [&](size_t count) {
        const size_t o = off;
        off = align256(off + count * es);
        return o;
    };
    const size_t o_tok = take(V * D), o_cls = take((size_t)(d.n_classes + 1) * D);
    std::vector<size_t> lo(L * 6);
    for (size_t l = 0; l < L; ++l) {
        lo[l * 6 + 0] = take(D);
        lo[l * 6 + 1] = take(3 * D * D);
        lo[l * 6 + 2] = take(D * D);
        lo[l * 6 + 3] = take(D);
        lo[l * 6 + 4] = take(2 * F * D);
        lo[l * 6 + 5] = take(D * F);
    }
    const size_t o_gout = take(D), o_head = take(V * D);
    if (off != weight_bytes) {
        snprintf(c->err, sizeof(c->err), "weight image is %zu bytes, the description needs %zu", weight_bytes, off);
        return HBSJD_EINVAL;
    }
    CK(cudaMalloc((void**)&c->w_img, off));
    CK(cudaMemcpyAsync(c->w_img, weights, off, cudaMemcpyHostToDevice, c->stream));
    if (c->bf16_model) {
        // RMSNorm is folded around the GEMMs: W' = W diag(gain), rounded to bf16 once (exact when the gain is 1).
        // Returns false when every gain is 1 and nothing has to be rewritten.
        auto bf2f = [](uint16_t b) {
            uint32_t u = (uint32_t)b << 16;
            float f;
            memcpy(&f, &u, 4);
            return f;
        };
        auto f2bf = [](float f) {
            uint32_t u;
            memcpy(&u, &f, 4);
            if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)(u >> 16);  // NaN
            return (uint16_t)((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
        };
        c->unit_gains = true;
        auto fold = [&](const uint16_t* W, const uint16_t* gain, size_t rows, std::vector<uint16_t>& out) {
            bool ones = true;
            for (size_t d = 0; d < D; ++d) ones = ones && gain[d] == 0x3f80;
            c->unit_gains = c->unit_gains && ones;
            if (ones || !c->fold_norm) return false;
            out.resize(rows * D);
            for (size_t r = 0; r < rows; ++r)
                for (size_t d = 0; d < D; ++d) out[r * D + d] = f2bf(bf2f(W[r * D + d]) * bf2f(gain[d]));
            return true;
        };
        const unsigned char* img = (const unsigned char*)weights;
        std::vector<uint16_t> tmp(2 * F * D), folded;
        for (size_t l = 0; l < L; ++l) {
            if (fold((const uint16_t*)(img + lo[l * 6 + 1]), (const uint16_t*)(img + lo[l * 6 + 0]), 3 * D, folded)) {
                CK(cudaMemcpyAsync(c->w_img + lo[l * 6 + 1], folded.data(), folded.size() * 2, cudaMemcpyHostToDevice,
                                   c->stream));
                CK(cudaStreamSynchronize(c->stream));
            }
            // the SwiGLU epilogue wants gate row f and up row f next to each other: rows (2f, 2f+1)
            const bool f13 = fold((const uint16_t*)(img + lo[l * 6 + 4]), (const uint16_t*)(img + lo[l * 6 + 3]), 2 * F,
                                  folded);
            const uint16_t* src = f13 ? folded.data() : (const uint16_t*)(img + lo[l * 6 + 4]);
            for (size_t f = 0; f < F; ++f) {
                memcpy(&tmp[(2 * f) * D], src + f * D, D * 2);
                memcpy(&tmp[(2 * f + 1) * D], src + (F + f) * D, D * 2);
            }
            CK(cudaMemcpyAsync(c->w_img + lo[l * 6 + 4], tmp.data(), tmp.size() * 2, cudaMemcpyHostToDevice,
                               c->stream));
            CK(cudaStreamSynchronize(c->stream));
        }
        if (fold((const uint16_t*)(img + o_head), (const uint16_t*)(img + o_gout), V, folded)) {
            CK(cudaMemcpyAsync(c->w_img + o_head, folded.data(), folded.size() * 2, cudaMemcpyHostToDevice, c->stream));
            CK(cudaStreamSynchronize(c->stream));
        }
    }
    c->tok_emb = c->w_img + o_tok;
    c->cls_emb = c->w_img + o_cls;
    c->g_out = c->w_img + o_gout;
    c->w_head = c->w_img + o_head;
    c->layers.resize(L);
    for (size_t l = 0; l < L; ++l) {
        c->layers[l].g_attn = c->w_img + lo[l * 6 + 0];
        c->layers[l].w_qkv = c->w_img + lo[l * 6 + 1];
        c->layers[l].w_o = c->w_img + lo[l * 6 + 2];
        c->layers[l].g_ffn = c->w_img + lo[l * 6 + 3];
        c->layers[l].w_13 = c->w_img + lo[l * 6 + 4];
        c->layers[l].w_2 = c->w_img + lo[l * 6 + 5];
    }
    // 2D rotary table by sequence index: index 0 unrotated; index s >= 1 at (row, col) of the raster
    {
        const int half = c->dh / 2, quarter = c->dh / 4;
        std::vector<float> tab((size_t)c->T * half * 2);
        for (int s = 0; s < c->T; ++s)
            for (int e = 0; e < half; ++e) {
                double ang = 0.0;
                if (s > 0) {
                    const int row = (s - 1) / d.grid_w, col = (s - 1) % d.grid_w;
                    const int ee = e < quarter ? e : e - quarter;
                    const double w = std::pow((double)d.rope_base, -(double)ee / (double)quarter);
                    ang = (e < quarter ? (double)row : (double)col) * w;
                }
                tab[((size_t)s * half + e) * 2] = (float)std::cos(ang);
                tab[((size_t)s * half + e) * 2 + 1] = (float)std::sin(ang);
            }
        CK(cudaMalloc((void**)&c->rope_cs, tab.size() * sizeof(float)));
        CK(cudaMemcpyAsync(c->rope_cs, tab.data(), tab.size() * sizeof(float), cudaMemcpyHostToDevice, c->stream));
        CK(cudaStreamSynchronize(c->stream));
    }
    // KV pages: two cache rows (conditional, unconditional) per image
    const int rows = 2 * c->Bmax;
    c->pages_per_row = (c->T + PAGE_TOKENS - 1) / PAGE_TOKENS;
    c->n_pages = rows * c->pages_per_row;
    const size_t kv_elems = L * (size_t)c->n_pages * PAGE_TOKENS * D;
    CK(cudaMalloc(&c->kc, kv_elems * es));
    CK(cudaMalloc(&c->vc, kv_elems * es));
    CK(cudaMemsetAsync(c->kc, 0, kv_elems * es, c->stream));
    CK(cudaMemsetAsync(c->vc, 0, kv_elems * es, c->stream));
    {
        std::vector<int32_t> tab(c->n_pages);
        for (int i = 0; i < c->n_pages; ++i) tab[i] = i;
        CK(cudaMalloc((void**)&c->page_table, tab.size() * sizeof(int32_t)));
        CK(cudaMemcpyAsync(c->page_table, tab.data(), tab.size() * sizeof(int32_t), cudaMemcpyHostToDevice,
                           c->stream));
        CK(cudaStreamSynchronize(c->stream));
    }
    // state
    const size_t Bm = c->Bmax, Wm = c->Wmax, T1 = c->T + 1;
    int rc;
    State& st = c->st;
    if ((rc = dev_alloc(c, &st.cursor, Bm)) || (rc = dev_alloc(c, &st.seq, Bm * T1)) ||
        (rc = dev_alloc(c, &st.delta, Bm * T1)) || (rc = dev_alloc(c, &st.qbase, Bm)) ||
        (rc = dev_alloc(c, &st.label, Bm)) || (rc = dev_alloc(c, &st.klen, Bm)) ||
        (rc = dev_alloc(c, &st.pfill, Bm)) || (rc = dev_alloc(c, &st.slot_img, Bm)) ||
        (rc = dev_alloc(c, &st.slot_c, Bm)) || (rc = dev_alloc(c, &st.slot_n, Bm)) ||
        (rc = dev_alloc(c, &st.slot_order, Bm)) ||
        (rc = dev_alloc(c, &st.counters, (size_t)8)) || (rc = dev_alloc(c, &st.m_last, Bm)) ||
        (rc = dev_alloc(c, &st.j_last, Bm)) || (rc = dev_alloc(c, &c->pbuf[0], Bm * Wm * V)) ||
        (rc = dev_alloc(c, &c->pbuf[1], Bm * Wm * V)) || (rc = dev_alloc(c, &c->flag, Bm * Wm)) ||
        (rc = dev_alloc(c, &c->cand_rep, Bm * Wm)) || (rc = dev_alloc(c, &c->cand_ref, Bm * Wm)))
        return rc;
    // activations for the largest forward: 2 branches x max_batch slots x max_window inputs
    const size_t Mmax = 2 * Bm * Wm;
    unsigned char *a, *q, *o, *act;
    const size_t f32_only = c->bf16_model ? 0 : 1;  // fp32 GEMM outputs the fused bf16 epilogues never materialise
    if ((rc = dev_alloc(c, &c->h, Mmax * D)) || (rc = dev_alloc(c, &c->qkv, f32_only * Mmax * 3 * D)) ||
        (rc = dev_alloc(c, &c->gu, f32_only * Mmax * 2 * F)) || (rc = dev_alloc(c, &c->logits, Mmax * V)) ||
        (rc = dev_alloc(c, &a, Mmax * D * es)) || (rc = dev_alloc(c, &q, Mmax * D * es)) ||
        (rc = dev_alloc(c, &o, Mmax * D * es)) || (rc = dev_alloc(c, &act, Mmax * F * es)))
        return rc;
    if ((rc = dev_alloc(c, &c->ssq, c->bf16_model ? Mmax * (D / 32) : (size_t)0))) return rc;
    c->a = a;
    c->q = q;
    c->o = o;
    c->act = act;
    if ((rc = dev_alloc(c, &c->stage_tok, Bm * (size_t)c->T)) || (rc = dev_alloc(c, &c->stage_len, Bm)) ||
        (rc = dev_alloc(c, &c->stage_lab, Bm)) || (rc = dev_alloc(c, &c->stage_out, Bm * (size_t)c->T)))
        return rc;
    {
        unsigned char* vs = nullptr;
        if ((rc = dev_alloc(c, &vs, verify_scratch_bytes(c->Bmax, c->Wmax)))) return rc;
        c->verify_scratch = vs;
        if ((rc = dev_alloc(c, &c->score_pos, (size_t)c->Bmax * c->T))) return rc;
        if ((rc = dev_alloc(c, &c->score_img, (size_t)c->Bmax))) return rc;
        if ((rc = dev_alloc(c, &c->score_loss, 1))) return rc;
        if ((rc = dev_alloc(c, &c->m_sync, 1))) return rc;
    }
    c->pool.resize(1024);
    for (auto& s : c->pool) {
        s.a = s.b = nullptr;
        CK(cudaEventCreate(&s.a));
        CK(cudaEventCreate(&s.b));
    }
    CK(cudaMallocHost((void**)&c->h_counters, 8 * sizeof(int32_t)));
    CK(cudaEventCreate(&c->ev0));
    CK(cudaEventCreate(&c->ev1));
    CK(cudaEventCreate(&c->ev2));
    CK(cudaStreamSynchronize(c->stream));
    return 0;
}

}  // namespace

extern "C" {

const char* hbsjd_strerror(int code) {
    switch (code) {
        case HBSJD_OK: return "ok";
        case HBSJD_EINVAL: return "invalid argument";
        case HBSJD_ENOMEM: return "out of memory";
        case HBSJD_ECUDA: return "CUDA error";
        case HBSJD_ESTATE: return "call not valid in this state";
        case HBSJD_ETIMEOUT: return "bounded device wait gave up";
        default: return "unknown error";
    }
}

const char* hbsjd_last_error(const hbsjd_ctx* c) { return c ? c->err : "null context"; }

int hbsjd_create(hbsjd_ctx** out, const hbsjd_model_desc* m, const void* weights, size_t weight_bytes,
                 int max_batch, int max_window, void* cuda_stream) {
    if (!out) return HBSJD_EINVAL;
    *out = nullptr;
    if (!m || !weights) return HBSJD_EINVAL;
    if (m->n_layers < 1 || m->dim < 16 || m->n_heads < 1 || m->dim % m->n_heads != 0 || m->ffn_hidden < 16 ||
        m->vocab < 4 || m->vocab % 4 != 0 || m->vocab > 32768 || m->grid_h < 1 || m->grid_w < 1 || m->n_classes < 1 ||
        (m->dtype != HBSJD_DTYPE_FP32 && m->dtype != HBSJD_DTYPE_BF16) || !(m->rms_eps > 0) || !(m->rope_base > 1) ||
        max_batch < 1 || max_window < 1 || max_window > 64)
        return HBSJD_EINVAL;
    const int dh = m->dim / m->n_heads;
    if (dh != 16 && dh != 32 && dh != 64 && dh != 128) return HBSJD_EINVAL;
    if (m->dim % 16 || m->ffn_hidden % 16) return HBSJD_EINVAL;
    // the fused QKV epilogue holds the cos/sin of at most 32 rotation pairs per row (head sizes 32 and 64)
    if (m->dtype == HBSJD_DTYPE_BF16 && (m->dim % 64 || m->ffn_hidden % 64 || m->vocab % 64 || (dh != 32 && dh != 64)))
        return HBSJD_EINVAL;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return HBSJD_ECUDA;
    hbsjd_ctx* c = new (std::nothrow) hbsjd_ctx();
    if (!c) return HBSJD_ENOMEM;
    memset((void*)&c->st, 0, sizeof(State));
    c->d = *m;
    c->T = m->grid_h * m->grid_w;
    c->dh = dh;
    c->Bmax = max_batch;
    c->Wmax = max_window;
    c->bf16_model = m->dtype == HBSJD_DTYPE_BF16;
    c->fold_norm = c->bf16_model && 2L * max_batch * max_window <= 2048;
    c->unit_gains = false;
    c->ref_attention = false;
    c->stream = (cudaStream_t)cuda_stream;
    c->dbg_layer = -1;
    c->err[0] = 0;
    const int rc = create_impl(c, weights, weight_bytes);
    if (rc != 0) {
        fprintf(stderr, "hbsjd_create: %s\n", c->err);
        free_all(c);
        delete c;
        return rc;
    }
    *out = c;
    return HBSJD_OK;
}

void hbsjd_destroy(hbsjd_ctx* c) {
    if (!c) return;
    cudaStreamSynchronize(c->stream);
    free_all(c);
    delete c;
}

int hbsjd_rollout(hbsjd_ctx* c, int batch, const int32_t* prefix_tokens, const int32_t* prefix_len,
                  const int32_t* class_labels, const hbsjd_params* p, int32_t* out_tokens, hbsjd_stats* stats) {
    if (!c) return HBSJD_EINVAL;
    c->err[0] = 0;
    if (!prefix_tokens || !prefix_len || !class_labels || !p || !out_tokens) {
        snprintf(c->err, sizeof(c->err), "null argument");
        return HBSJD_EINVAL;
    }
    if (batch < 1 || batch > c->Bmax || p->window < 1 || p->window > c->Wmax || p->history_offset < 1 ||
        !(p->temperature > 0.f) || !std::isfinite(p->cfg_scale) || p->top_k < 0 ||
        (p->verify_mode != HBSJD_VERIFY_PROB && p->verify_mode != HBSJD_VERIFY_GREEDY) ||
        p->exec_mode < HBSJD_EXEC_FULL || p->exec_mode > HBSJD_EXEC_SYNC || p->gamma < 0) {
        snprintf(c->err, sizeof(c->err), "parameter out of range (batch %d window %d)", batch, p->window);
        return HBSJD_EINVAL;
    }
    const int T = c->T, V = c->d.vocab;
    // validate the integer inputs on the host before any kernel runs
    std::vector<int32_t> hk(batch), hl(batch), ht((size_t)batch * T);
    CK(cudaMemcpyAsync(hk.data(), prefix_len, batch * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(hl.data(), class_labels, batch * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(ht.data(), prefix_tokens, (size_t)batch * T * sizeof(int32_t), cudaMemcpyDeviceToHost,
                       c->stream));
    CK(cudaStreamSynchronize(c->stream));
    int kmax = 0, live = 0;
    for (int b = 0; b < batch; ++b) {
        if (hk[b] < 0 || hk[b] > T || hl[b] < 0 || hl[b] > c->d.n_classes) {
            snprintf(c->err, sizeof(c->err), "image %d: prefix_len %d or label %d out of range", b, hk[b], hl[b]);
            return HBSJD_EINVAL;
        }
        for (int t = 0; t < hk[b]; ++t)
            if (ht[(size_t)b * T + t] < 0 || ht[(size_t)b * T + t] >= V) {
                snprintf(c->err, sizeof(c->err), "image %d: prefix token %d out of range", b, t);
                return HBSJD_EINVAL;
            }
        kmax = hk[b] > kmax ? hk[b] : kmax;
        live += hk[b] < T;
    }
    c->P = *p;
    State& st = c->st;
    st.B = batch;
    st.T = T;
    st.V = V;
    st.D = c->d.dim;
    st.Hh = c->d.n_heads;
    st.dh = c->dh;
    st.F = c->d.ffn_hidden;
    st.L = c->d.n_layers;
    st.C = c->d.n_classes;
    st.Bmax = c->Bmax;
    st.Wmax = c->Wmax;
    st.W = p->window;
    st.H = p->history_offset;
    st.nb = p->cfg_scale != 1.0f ? 2 : 1;
    memset(&c->stats, 0, sizeof(c->stats));
    c->launches = 0;
    c->round = 0;
    c->parity = 0;
    c->live = live;
    c->have_rollout = false;

    CK(cudaEventRecord(c->ev0, c->stream));
    launch_init_state(st, prefix_tokens, prefix_len, class_labels, c->stream);
    c->launches++;
    // prefix pre-filling: cache sequence indices 0..k-1 in chunks of W (no LM head)
    for (int pr = 0;; ++pr) {
        int act = 0;
        for (int b = 0; b < batch; ++b) act += hk[b] > pr * p->window;
        if (act == 0) break;
        const int compact = choose_compact(c, act);
        const int S = compact ? act : batch;
        launch_setup(st, 1, compact, c->stream);
        const int rc = forward_any(c, S, false);
        if (rc) return rc;
        launch_prefill_advance(st, S, c->stream);
        c->launches += 2;
        c->stats.prefill_forwards += 1;
        if (c->profiling) {  // fold this forward's event pairs while its byte counters are current
            const int rs = sync_counters(c);
            if (rs) return rs;
        }
    }
    launch_init_window(st, (uint32_t)(p->seed & 0xffffffffu), (uint32_t)(p->seed >> 32), c->stream);
    c->launches++;
    CK(cudaEventRecord(c->ev1, c->stream));
    if (c->profiling) {
        const int rc = sync_counters(c);
        if (rc) return rc;
    }
    CK(cudaGetLastError());
    c->have_rollout = true;

    int rounds = 0;
    while (c->live > 0 && (p->max_rounds < 0 || rounds < p->max_rounds)) {
        const int rc = run_round(c);
        if (rc) return rc;
        ++rounds;
    }
    launch_export_tokens(st, out_tokens, c->stream);
    c->launches++;
    CK(cudaEventRecord(c->ev2, c->stream));
    const int rc = sync_counters(c);
    if (rc) return rc;
    CK(cudaEventElapsedTime(&c->stats.ms_prefill, c->ev0, c->ev1));
    CK(cudaEventElapsedTime(&c->stats.ms_total, c->ev0, c->ev2));
    c->stats.kernel_launches = c->launches;
    if (stats) *stats = c->stats;
    return HBSJD_OK;
}

int hbsjd_rollout_host(hbsjd_ctx* c, int batch, const int32_t* prefix_tokens, const int32_t* prefix_len,
                       const int32_t* class_labels, const hbsjd_params* p, int32_t* out_tokens, hbsjd_stats* stats) {
    if (!c) return HBSJD_EINVAL;
    if (!prefix_tokens || !prefix_len || !class_labels || !p || !out_tokens || batch < 1 || batch > c->Bmax) {
        snprintf(c->err, sizeof(c->err), "null argument or batch out of range");
        return HBSJD_EINVAL;
    }
    const size_t bt = (size_t)batch * c->T * sizeof(int32_t), bb = (size_t)batch * sizeof(int32_t);
    CK(cudaMemcpyAsync(c->stage_tok, prefix_tokens, bt, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(c->stage_len, prefix_len, bb, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(c->stage_lab, class_labels, bb, cudaMemcpyHostToDevice, c->stream));
    const int rc = hbsjd_rollout(c, batch, c->stage_tok, c->stage_len, c->stage_lab, p, c->stage_out, stats);
    if (rc) return rc;
    CK(cudaMemcpyAsync(out_tokens, c->stage_out, bt, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBSJD_OK;
}

int hbsjd_probs(hbsjd_ctx* c, const float* logits_c, const float* logits_u, int rows, float cfg_scale,
                float temperature, int top_k, float* probs) {
    if (!c || !logits_c || !probs || rows < 1 || !(temperature > 0.f) || top_k < 0 ||
        (((uintptr_t)logits_c | (uintptr_t)logits_u | (uintptr_t)probs) & 15))
        return HBSJD_EINVAL;
    launch_probs(logits_c, logits_u, rows, c->d.vocab, cfg_scale, temperature, top_k, probs, c->stream);
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(c->stream));
    return HBSJD_OK;
}

int hbsjd_verify(hbsjd_ctx* c, const hbsjd_verify_desc* d, const float* logits, const float* q_prev, float* p_out,
                 int32_t* cursor, int32_t* seq, uint8_t* delta, int32_t* qbase, int32_t* m_out) {
    if (!c) return HBSJD_EINVAL;
    if (!d || !logits || !q_prev || !p_out || !cursor || !seq || !delta || !qbase || !m_out || d->batch < 1 ||
        d->batch > c->Bmax || d->window < 1 || d->window > c->Wmax || d->T < 1 || d->V < 4 || d->V % 4 ||
        d->V > 32768 || (d->branches != 1 && d->branches != 2) || d->history_offset < 1 ||
        !(d->temperature > 0.f) || !std::isfinite(d->temperature) || !std::isfinite(d->cfg_scale) || d->top_k < 0) {
        snprintf(c->err, sizeof(c->err), "hbsjd_verify: argument out of range");
        return HBSJD_EINVAL;
    }
    static_assert(sizeof(VerifyDesc) == sizeof(hbsjd_verify_desc), "descriptor layouts must agree");
    VerifyDesc vd;
    memcpy(&vd, d, sizeof(vd));
    const VerifyScratch sc = verify_scratch_carve(c->verify_scratch, d->batch, d->window);
    CK(verify_enqueue(vd, sc, logits, q_prev, p_out, cursor, seq, delta, qbase, m_out, c->stream));
    // the kernels check the caller's state arrays as they read them (cursor, draft tokens, proposal rows): a
    // value that cannot be valid is recorded, its access skipped, and reported here
    int32_t code = 0;
    CK(cudaMemcpyAsync(&code, sc.counters + CNT_ERROR, sizeof(code), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (code != 0) {
        snprintf(c->err, sizeof(c->err), "hbsjd_verify: invalid state array on the device (code %d)", code);
        return code >= 16 ? HBSJD_EINVAL : HBSJD_ETIMEOUT;
    }
    return HBSJD_OK;
}

int hbsjd_bikl(hbsjd_ctx* c, const float* logits_s, const float* logits_t, int rows, float* out) {
    if (!c) return HBSJD_EINVAL;
    if (!logits_s || !logits_t || !out || rows < 1 || c->d.vocab % 4) {
        snprintf(c->err, sizeof(c->err), "hbsjd_bikl: argument out of range");
        return HBSJD_EINVAL;
    }
    launch_bikl_rows(logits_s, logits_t, rows, c->d.vocab, out, c->stream);
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(c->stream));
    return HBSJD_OK;
}

int hbsjd_score(hbsjd_ctx* student, hbsjd_ctx* teacher, int batch, const int32_t* tokens, const int32_t* prefix_len,
                const int32_t* class_labels, float* bikl_pos, float* per_image, float* loss) {
    hbsjd_ctx* c = student;  // errors are reported on the student context
    if (!c) return HBSJD_EINVAL;
    c->err[0] = 0;
    if (!teacher || teacher == student || !tokens || !prefix_len || !class_labels || !loss) {
        snprintf(c->err, sizeof(c->err), "hbsjd_score: null argument, or one context given twice");
        return HBSJD_EINVAL;
    }
    const int T = c->T, V = c->d.vocab;
    if (teacher->T != T || teacher->d.vocab != V || teacher->d.grid_w != c->d.grid_w || V % 4 || batch < 1 ||
        batch > c->Bmax || batch > teacher->Bmax || teacher->d.n_classes != c->d.n_classes) {
        snprintf(c->err, sizeof(c->err), "hbsjd_score: contexts do not match (grid, vocabulary, classes) or batch %d too large",
                 batch);
        return HBSJD_EINVAL;
    }
    // validate the integer inputs on the host before any kernel runs
    std::vector<int32_t> hk(batch), hl(batch), ht((size_t)batch * T);
    CK(cudaMemcpyAsync(hk.data(), prefix_len, batch * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(hl.data(), class_labels, batch * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(ht.data(), tokens, (size_t)batch * T * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    for (int b = 0; b < batch; ++b) {
        if (hk[b] < 0 || hk[b] > T || hl[b] < 0 || hl[b] > c->d.n_classes) {
            snprintf(c->err, sizeof(c->err), "image %d: prefix_len %d or label %d out of range", b, hk[b], hl[b]);
            return HBSJD_EINVAL;
        }
        for (int t = 0; t < T; ++t)
            if (ht[(size_t)b * T + t] < 0 || ht[(size_t)b * T + t] >= V) {
                snprintf(c->err, sizeof(c->err), "image %d: token %d out of range", b, t);
                return HBSJD_EINVAL;
            }
    }
    // inputs per image per chunk: one branch only, so the activation buffers (sized for two branches of
    // max_window inputs) hold twice the rollout's window
    int W = 2 * (c->Wmax < teacher->Wmax ? c->Wmax : teacher->Wmax);
    if (W > 64) W = 64;
    if (W > T) W = T;
    float* pos = bikl_pos ? bikl_pos : c->score_pos;
    float* img = per_image ? per_image : c->score_img;
    hbsjd_ctx* both[2] = {student, teacher};
    for (hbsjd_ctx* x : both) {
        State& st = x->st;
        st.B = batch;
        st.T = T;
        st.V = V;
        st.D = x->d.dim;
        st.Hh = x->d.n_heads;
        st.dh = x->dh;
        st.F = x->d.ffn_hidden;
        st.L = x->d.n_layers;
        st.C = x->d.n_classes;
        st.Bmax = x->Bmax;
        st.Wmax = x->Wmax;
        st.W = W;
        st.H = 1;
        st.nb = 1;
        x->have_rollout = false;
        x->live = 0;
        launch_score_init(st, tokens, class_labels, prefix_len, x == student ? pos : nullptr, x->stream);
        x->launches++;
    }
    for (int done = 0; done < T; done += W) {
        for (hbsjd_ctx* x : both) {
            launch_setup(x->st, 1, 0, x->stream);
            x->launches++;
            const int rc = forward_any(x, batch, true);
            if (rc) {
                if (x != c) snprintf(c->err, sizeof(c->err), "teacher forward: %.200s", x->err);
                return rc;
            }
            if (x->profiling) {  // fold this forward's event pairs while its byte counters are current
                const int rs = sync_counters(x);
                if (rs) return rs;
            }
        }
        // the divergence kernel reads both models' logits on the student's stream; the teacher's next
        // forward overwrites its logits and waits for that kernel in turn
        CK(cudaEventRecord(teacher->ev2, teacher->stream));
        CK(cudaStreamWaitEvent(c->stream, teacher->ev2, 0));
        {
            // timed with the vocabulary-wide class: 2 V floats read per input, as the byte count of that class
            const int ps = prof_begin(c, HBSJD_PROF_ACCEPT, 0.0);
            launch_bikl_slots(c->st, batch, c->logits, teacher->logits, prefix_len, pos, c->stream);
            prof_end(c, ps);
        }
        c->launches++;
        CK(cudaEventRecord(c->ev2, c->stream));
        CK(cudaStreamWaitEvent(teacher->stream, c->ev2, 0));
        for (hbsjd_ctx* x : both) {
            launch_prefill_advance(x->st, batch, x->stream);
            x->launches++;
        }
    }
    launch_score_reduce(batch, T, prefix_len, pos, img, c->score_loss, c->stream);
    c->launches++;
    CK(cudaMemcpyAsync(loss, c->score_loss, sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaGetLastError());
    for (hbsjd_ctx* x : both) {
        const int rc = sync_counters(x);
        if (rc) {
            if (x != c) snprintf(c->err, sizeof(c->err), "teacher: %.200s", x->err);
            return rc;
        }
    }
    return HBSJD_OK;
}

int hbsjd_profile(hbsjd_ctx* c, int enable) {
    if (!c) return HBSJD_EINVAL;
    CK(cudaStreamSynchronize(c->stream));
    c->profiling = enable != 0;
    c->pool_used = 0;
    if (enable) memset(&c->prof, 0, sizeof(c->prof));  // switching off keeps the totals readable
    return HBSJD_OK;
}

int hbsjd_profile_read(hbsjd_ctx* c, hbsjd_kernel_profile* out) {
    if (!c || !out) return HBSJD_EINVAL;
    *out = c->prof;
    return HBSJD_OK;
}

int hbsjd_profile_launch_floor(hbsjd_ctx* c, int reps, float* us_out) {
    if (!c) return HBSJD_EINVAL;
    if (!us_out || reps < 1 || reps > (int)c->pool.size()) {
        snprintf(c->err, sizeof(c->err), "hbsjd_profile_launch_floor: argument out of range");
        return HBSJD_EINVAL;
    }
    CK(cudaStreamSynchronize(c->stream));
    // a kernel in front, so that every bracket starts behind a completed kernel as in a forward
    launch_noop(c->stream);
    for (int i = 0; i < reps; ++i) {
        CK(cudaEventRecord(c->pool[i].a, c->stream));
        launch_noop(c->stream);
        CK(cudaEventRecord(c->pool[i].b, c->stream));
    }
    CK(cudaStreamSynchronize(c->stream));
    std::vector<float> us(reps);
    for (int i = 0; i < reps; ++i) {
        float ms = 0.f;
        CK(cudaEventElapsedTime(&ms, c->pool[i].a, c->pool[i].b));
        us[i] = ms * 1e3f;
    }
    std::sort(us.begin(), us.end());
    *us_out = us[reps / 2];
    return HBSJD_OK;
}

int hbsjd_calibrate_gamma(hbsjd_ctx* c, int batch, int window, int guidance, int* gamma_out, float* ms_full,
                          float* ms_compact) {
    if (!c) return HBSJD_EINVAL;
    if (!gamma_out || batch < 1 || batch > c->Bmax || window < 1 || window > c->Wmax) {
        snprintf(c->err, sizeof(c->err), "hbsjd_calibrate_gamma: argument out of range");
        return HBSJD_EINVAL;
    }
    c->have_rollout = false;
    State& st = c->st;
    st.B = batch;
    st.T = c->T;
    st.V = c->d.vocab;
    st.D = c->d.dim;
    st.Hh = c->d.n_heads;
    st.dh = c->dh;
    st.F = c->d.ffn_hidden;
    st.L = c->d.n_layers;
    st.C = c->d.n_classes;
    st.Bmax = c->Bmax;
    st.Wmax = c->Wmax;
    st.W = window;
    st.H = 1;
    st.nb = guidance ? 2 : 1;
    const int points[5] = {batch, (3 * batch) / 4, batch / 2, batch / 4, batch / 8};
    int gamma = 0;
    for (int p = 0; p < 5; ++p) {
        const int live = points[p] < 1 ? 1 : points[p];
        float best[2] = {0.f, 0.f};
        for (int compact = 0; compact < 2; ++compact) {
            const int S = compact ? live : batch;
            for (int rep = 0; rep < 4; ++rep) {  // the first repetition warms up
                launch_calib_state(st, live, c->stream);
                launch_setup(st, 0, compact, c->stream);
                CK(cudaEventRecord(c->ev0, c->stream));
                const int rc = forward_any(c, S, true);
                if (rc) return rc;
                CK(cudaEventRecord(c->ev1, c->stream));
                const int rs = sync_counters(c);
                if (rs) return rs;
                float ms = 0.f;
                CK(cudaEventElapsedTime(&ms, c->ev0, c->ev1));
                if (rep > 0 && (best[compact] == 0.f || ms < best[compact])) best[compact] = ms;
            }
        }
        if (ms_full) ms_full[p] = best[0];
        if (ms_compact) ms_compact[p] = best[1];
        if (best[1] <= best[0] * 1.01f && live > gamma) gamma = live;  // 1 % timing noise
    }
    *gamma_out = gamma;
    return HBSJD_OK;
}

int hbsjd_round(hbsjd_ctx* c, int* live_out) {
    if (!c) return HBSJD_EINVAL;
    if (!c->have_rollout) {
        snprintf(c->err, sizeof(c->err), "hbsjd_round needs a preceding hbsjd_rollout");
        return HBSJD_ESTATE;
    }
    const int rc = run_round(c);
    if (rc) return rc;
    if (live_out) *live_out = c->live;
    return HBSJD_OK;
}

int hbsjd_tokens(hbsjd_ctx* c, int32_t* out_tokens) {
    if (!c || !out_tokens) return HBSJD_EINVAL;
    if (!c->have_rollout) return HBSJD_ESTATE;
    launch_export_tokens(c->st, out_tokens, c->stream);
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(c->stream));
    return HBSJD_OK;
}

int hbsjd_get_state(hbsjd_ctx* c, int32_t* cursor, int32_t* seq, uint8_t* delta, int32_t* qbase, int32_t* round) {
    if (!c) return HBSJD_EINVAL;
    if (!c->have_rollout) return HBSJD_ESTATE;
    const size_t B = c->st.B, T1 = c->T + 1;
    if (cursor) CK(cudaMemcpyAsync(cursor, c->st.cursor, B * 4, cudaMemcpyDeviceToHost, c->stream));
    if (seq) CK(cudaMemcpyAsync(seq, c->st.seq, B * T1 * 4, cudaMemcpyDeviceToHost, c->stream));
    if (delta) CK(cudaMemcpyAsync(delta, c->st.delta, B * T1, cudaMemcpyDeviceToHost, c->stream));
    if (qbase) CK(cudaMemcpyAsync(qbase, c->st.qbase, B * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (round) *round = c->round;
    return HBSJD_OK;
}

int hbsjd_set_state(hbsjd_ctx* c, const int32_t* cursor, const int32_t* seq, const uint8_t* delta,
                    const int32_t* qbase, int32_t round) {
    if (!c || !cursor || !seq || !delta || !qbase) return HBSJD_EINVAL;
    if (!c->have_rollout) return HBSJD_ESTATE;
    const size_t B = c->st.B, T1 = c->T + 1;
    int live = 0;
    for (size_t b = 0; b < B; ++b) {
        if (cursor[b] < 0 || cursor[b] > c->T || qbase[b] < 0 || qbase[b] > cursor[b]) {
            snprintf(c->err, sizeof(c->err), "set_state: image %zu cursor/qbase out of range", b);
            return HBSJD_EINVAL;
        }
        for (size_t t = 1; t < T1; ++t)
            if (seq[b * T1 + t] < 0 || seq[b * T1 + t] >= c->d.vocab) {
                snprintf(c->err, sizeof(c->err), "set_state: image %zu token %zu out of range", b, t);
                return HBSJD_EINVAL;
            }
        // a sampled draft (delta = 0) at position t reads row t - qbase - 1 of the previous round's probabilities
        for (int t = cursor[b] + 1; t < cursor[b] + c->st.W && t < c->T; ++t)
            if (!delta[b * T1 + t] && t - qbase[b] - 1 >= c->Wmax) {
                snprintf(c->err, sizeof(c->err), "set_state: image %zu draft %d has no proposal row", b, t);
                return HBSJD_EINVAL;
            }
        live += cursor[b] < c->T;
    }
    CK(cudaMemcpyAsync(c->st.cursor, cursor, B * 4, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(c->st.seq, seq, B * T1 * 4, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(c->st.delta, delta, B * T1, cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(c->st.qbase, qbase, B * 4, cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    c->live = live;
    c->round = round;
    return HBSJD_OK;
}

int hbsjd_debug_forward(hbsjd_ctx* c, int layer, int stage) {
    if (!c) return HBSJD_EINVAL;
    if (!c->have_rollout) return HBSJD_ESTATE;
    if (layer < 0 || layer >= c->d.n_layers || (stage != 0 && stage != 1)) {
        snprintf(c->err, sizeof(c->err), "hbsjd_debug_forward: layer or stage out of range");
        return HBSJD_EINVAL;
    }
    launch_setup(c->st, 0, 0, c->stream);
    const int rc = forward_any(c, c->st.B, false, layer, stage);
    if (rc) return rc;
    CK(cudaGetLastError());
    c->last_S = c->st.B;
    c->last_compact = 0;
    c->dbg_layer = layer;
    return sync_counters(c);
}

int hbsjd_debug_read(hbsjd_ctx* c, int what, int index, void* host_dst, size_t max_bytes) {
    if (!c || !host_dst) return HBSJD_EINVAL;
    if (!c->have_rollout || (c->round == 0 && c->dbg_layer < 0)) return HBSJD_ESTATE;
    const int S = c->last_S, W = c->st.W, V = c->d.vocab;
    std::vector<int32_t> slots((size_t)3 * S);
    CK(cudaMemcpyAsync(slots.data(), c->st.slot_img, S * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(slots.data() + S, c->st.slot_c, S * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaMemcpyAsync(slots.data() + 2 * S, c->st.slot_n, S * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (what == HBSJD_DBG_SLOTS) {
        if (max_bytes < slots.size() * 4) return HBSJD_EINVAL;
        memcpy(host_dst, slots.data(), slots.size() * 4);
        return S;
    }
    const int img = what == HBSJD_DBG_PROBS ? index : index / 2;
    const int branch = what == HBSJD_DBG_PROBS ? 0 : index % 2;
    if (img < 0 || img >= c->st.B || (branch == 1 && c->st.nb == 1)) return HBSJD_EINVAL;
    int slot = -1;
    for (int s = 0; s < S; ++s)
        if (slots[s] == img) slot = s;
    if (slot < 0) return 0;
    const int n = slots[2 * S + slot];
    if (n == 0) return 0;
    if (what >= HBSJD_DBG_ACT_A && what <= HBSJD_DBG_ACT_H) {
        // rows of the slot in an activation buffer, as the last (partial) forward left them
        const size_t es = c->bf16_model ? 2 : 4, D = c->d.dim, F = c->d.ffn_hidden;
        const size_t row0 = (size_t)(branch * S + slot) * W;
        const unsigned char* src;
        size_t width;
        switch (what) {
            case HBSJD_DBG_ACT_A: src = (const unsigned char*)c->a; width = D * es; break;
            case HBSJD_DBG_ACT_Q: src = (const unsigned char*)c->q; width = D * es; break;
            case HBSJD_DBG_ACT_O: src = (const unsigned char*)c->o; width = D * es; break;
            case HBSJD_DBG_ACT_FFN: src = (const unsigned char*)c->act; width = F * es; break;
            default: src = (const unsigned char*)c->h; width = D * 4; break;
        }
        if (max_bytes < (size_t)n * width) return HBSJD_EINVAL;
        CK(cudaMemcpyAsync(host_dst, src + row0 * width, (size_t)n * width, cudaMemcpyDeviceToHost, c->stream));
        CK(cudaStreamSynchronize(c->stream));
        return n;
    }
    if (what == HBSJD_DBG_KV_K || what == HBSJD_DBG_KV_V) {
        // cache rows of sequence indices 0 .. c+n-1 of the layer of the last hbsjd_debug_forward
        if (c->dbg_layer < 0) return HBSJD_ESTATE;
        const size_t es = c->bf16_model ? 2 : 4, D = c->d.dim;
        const int rows = slots[S + slot] + n;
        if (max_bytes < (size_t)rows * D * es) return HBSJD_EINVAL;
        std::vector<int32_t> pt(c->pages_per_row);
        const int crow = branch * c->Bmax + img;
        CK(cudaMemcpyAsync(pt.data(), c->page_table + (size_t)crow * c->pages_per_row, pt.size() * 4,
                           cudaMemcpyDeviceToHost, c->stream));
        CK(cudaStreamSynchronize(c->stream));
        const unsigned char* pool = (const unsigned char*)(what == HBSJD_DBG_KV_K ? c->kc : c->vc);
        for (int s0 = 0; s0 < rows; s0 += PAGE_TOKENS) {
            const int cnt = rows - s0 < PAGE_TOKENS ? rows - s0 : PAGE_TOKENS;
            const size_t off = (((size_t)c->dbg_layer * c->n_pages + pt[s0 / PAGE_TOKENS]) * PAGE_TOKENS) * D * es;
            CK(cudaMemcpyAsync((unsigned char*)host_dst + (size_t)s0 * D * es, pool + off, (size_t)cnt * D * es,
                               cudaMemcpyDeviceToHost, c->stream));
        }
        CK(cudaStreamSynchronize(c->stream));
        return rows;
    }
    const size_t bytes = (size_t)n * V * sizeof(float);
    if (max_bytes < bytes) return HBSJD_EINVAL;
    const float* src;
    if (what == HBSJD_DBG_PROBS) src = c->pbuf[c->parity ^ 1] + (size_t)img * c->Wmax * V;
    else if (what == HBSJD_DBG_LOGITS) src = c->logits + ((size_t)(branch * S + slot) * W) * V;
    else return HBSJD_EINVAL;
    CK(cudaMemcpyAsync(host_dst, src, bytes, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return n;
}

int hbsjd_gemm(hbsjd_ctx* c, const void* A, const void* W, float* C, int M, int N, int K, int accumulate) {
    return hbsjd_debug_gemm(c, A, W, C, M, N, K, accumulate, 1, 0, 0);
}

int hbsjd_debug_gemm(hbsjd_ctx* c, const void* A, const void* W, float* C, int M, int N, int K, int accumulate,
                     int reps, unsigned int acc_wait_ns, int tile) {
    if (!c || !A || !W || !C || M < 1 || N < 1 || K < 1 || reps < 1) return HBSJD_EINVAL;
    if (accumulate == 2 && (!c->bf16_model || N != c->d.dim || M > 2 * c->Bmax * c->Wmax)) {
        snprintf(c->err, sizeof(c->err), "hbsjd_debug_gemm: the residual-update form needs a bf16 context, N = dim and "
                                         "M within the context's activation rows");
        return HBSJD_EINVAL;
    }
    for (int r = 0; r < reps; ++r) {
        int rc;
        if (accumulate == 2) {
            // the form the forward uses for its residual updates: C += A W^T, plus the bf16 copy and the partial
            // sums of squares of the new rows (into the context's own buffers)
            c->launches++;
            rc = gemm_tcgen05_addnorm((const bf16*)A, (const bf16*)W, C, (bf16*)c->a, c->ssq, M, N, K, 0,
                                      c->st.counters + CNT_ERROR, c->stream, c->err, sizeof(c->err));
            if (rc) rc = rc == -1 ? HBSJD_EINVAL : HBSJD_ECUDA;
        } else {
            // W is the caller's buffer, possibly written by earlier work of the stream: no early fetch of its tiles
            rc = c->bf16_model ? gemm<bf16>(c, A, W, C, M, N, K, accumulate, 0, 0, acc_wait_ns, tile)
                               : gemm<float>(c, A, W, C, M, N, K, accumulate);
        }
        if (rc) return rc;
    }
    CK(cudaGetLastError());
    return sync_counters(c);
}

int hbsjd_debug_fold_norm(hbsjd_ctx* c, int on) {
    if (!c) return HBSJD_EINVAL;
    if (!c->bf16_model || c->have_rollout || !c->unit_gains) {
        snprintf(c->err, sizeof(c->err), "hbsjd_debug_fold_norm: needs a bf16 context with unit norm gains, before its "
                                         "first rollout");
        return HBSJD_ESTATE;
    }
    c->fold_norm = on != 0;
    return HBSJD_OK;
}

int hbsjd_debug_shuffle_pages(hbsjd_ctx* c, uint64_t seed) {
    if (!c) return HBSJD_EINVAL;
    if (c->have_rollout) {
        snprintf(c->err, sizeof(c->err), "hbsjd_debug_shuffle_pages: only before the first rollout of the context");
        return HBSJD_ESTATE;
    }
    std::vector<int32_t> tab(c->n_pages);
    for (int i = 0; i < c->n_pages; ++i) tab[i] = i;
    uint64_t x = 0x9E3779B97F4A7C15ull * (seed | 1ull);
    for (int i = c->n_pages - 1; i > 0; --i) {
        x = x * 6364136223846793005ull + 1442695040888963407ull;
        const int j = (int)((x >> 33) % (uint64_t)(i + 1));
        std::swap(tab[i], tab[j]);
    }
    CK(cudaMemcpyAsync(c->page_table, tab.data(), tab.size() * sizeof(int32_t), cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBSJD_OK;
}

}  // extern "C"
