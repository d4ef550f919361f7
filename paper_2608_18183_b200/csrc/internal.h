// Launchers of the rollout kernels (internal to the library; the public boundary is include/hbsjd.h).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "common.cuh"

struct CUtensorMap_st;  // CUtensorMap of <cuda.h>

namespace hbsjd {

// Device-side rollout state and per-round slot tables.  A "slot" is the place of one image in the
// physical batch of a forward: Full execution has one slot per image of the batch (finished images
// get n = 0), Compact execution one slot per live image.  Token row of (branch, slot, i) =
// (branch * S + slot) * W + i.
struct State {
    int B, T, V, D, Hh, dh, F, L, C;  // batch, tokens per image, vocab, dim, heads, head dim, ffn, layers, classes
    int Bmax, Wmax;
    int W, H;        // window (inputs per image per round), history offset
    int nb;          // branches: 1, or 2 under classifier-free guidance
    int32_t* cursor;   // [Bmax] committed tokens
    int32_t* seq;      // [Bmax][T+1] tokens by 1-based position (committed, then drafts)
    uint8_t* delta;    // [Bmax][T+1] draft carries a point-mass proposal
    int32_t* qbase;    // [Bmax] cursor at the start of the previous round
    int32_t* label;    // [Bmax]
    int32_t* klen;     // [Bmax] prefix length
    int32_t* pfill;    // [Bmax] prefill cursor
    int32_t* slot_img; // [Bmax]
    int32_t* slot_c;   // [Bmax] first sequence index of the slot's inputs
    int32_t* slot_n;   // [Bmax] number of inputs (0: inactive slot)
    int32_t* slot_order;  // [Bmax] slots by context length c + n, longest first (null: not built)
    int32_t* counters; // [8], see CNT_*
    int32_t* m_last;   // [Bmax] tokens committed in the last round
    int32_t* j_last;   // [Bmax] first-reject index of the last round (-1 none)
};

enum { CNT_LIVE = 0, CNT_COMMITTED = 1, CNT_REJECTS = 2, CNT_LIVE_SETUP = 3, CNT_SLOTS = 4, CNT_ERROR = 5,
       CNT_SUM_KEYS = 6 /* sum over active slots of c+n */, CNT_SUM_N = 7 /* sum of n */ };

struct AcceptArgs {
    const float* logits;  // [nb][S][W][V]
    float* pcur;          // [Bmax][Wmax][V] this round's probabilities (next round's proposals)
    const float* pprev;   // [Bmax][Wmax][V]
    uint8_t* flag;        // [Bmax][Wmax] 1 = draft accepted
    int32_t* cand_rep;    // [Bmax][Wmax] replacement (or bonus) token candidate of position i
    int32_t* cand_ref;    // [Bmax][Wmax] refreshed draft candidate of position i
    int S;
    float cfg_scale, temperature;
    int top_k, greedy;
    uint32_t seed_lo, seed_hi, round;
    const int32_t* m_sync;  // batch-synchronous progress: the smallest commit of the batch (null: independent)
};

// ---- row operations (model_kernels.cu)
void launch_setup(const State& st, int phase /*0 round, 1 prefill*/, int compact, cudaStream_t s);
// hb / ssq (bf16 model, may be null): the bf16 copy of the embedded rows and their partial sums of squares per
// 32-column chunk, as the folded RMSNorm of the first projection wants them
template <typename TA>
void launch_embed(const State& st, int S, const TA* tok_emb, const TA* cls_emb, float* h, bf16* hb, float* ssq,
                  cudaStream_t s);
template <typename TA>
void launch_rmsnorm(const float* h, const TA* gain, TA* out, int M, int D, float eps, cudaStream_t s);
template <typename TA>
void launch_rope_kv(const State& st, int S, int layer, const float* qkv, const float* rope_cs, TA* q, KvView kv,
                    cudaStream_t s);
template <typename TA>
void launch_attention_ref(const State& st, int S, int layer, const TA* q, KvView kv, TA* out, cudaStream_t s);
template <typename TA>
void launch_swiglu(const float* gu, TA* act, int M, int F, cudaStream_t s);
template <typename TA>
void launch_gemm_simt(const TA* A, const TA* W, float* C, int M, int N, int K, int accumulate, cudaStream_t s);

// Scratch of the stand-alone verification step, carved from one allocation.
struct VerifyScratch {
    int32_t *slot_img, *slot_c, *slot_n, *j_last, *counters;
    uint8_t* flag;
    int32_t *cand_rep, *cand_ref;
};
size_t verify_scratch_bytes(int batch, int window);
VerifyScratch verify_scratch_carve(void* base, int batch, int window);
struct VerifyDesc {  // mirrors hbsjd_verify_desc
    int32_t batch, window, T, V, branches, history_offset, greedy, top_k;
    float cfg_scale, temperature;
    uint64_t seed;
    uint32_t round, reserved;
};
// Enqueues set-up, probability/accept and commit kernels on caller state with the given scratch.
cudaError_t verify_enqueue(const VerifyDesc& d, const VerifyScratch& sc, const float* logits, const float* q_prev,
                           float* p_out, int32_t* cursor, int32_t* seq, uint8_t* delta, int32_t* qbase,
                           int32_t* m_out, cudaStream_t s);

// ---- persistent tensor-core ragged attention, bf16, head size 64 (attention_tma.cu)
bool attention_tma_supported(const State& st, const KvView& kv);
// q_rows_cap: row capacity of the q buffer.  Returns 0 or a negative code with a message in err.
int launch_attention_tma(const State& st, int S, int layer, const bf16* q, int q_rows_cap, KvView kv, bf16* out,
                         int32_t* error_flag, cudaStream_t s, char* err, size_t errlen);

// ---- state kernels (state_kernels.cu)
void launch_init_state(const State& st, const int32_t* prefix_tokens, const int32_t* prefix_len,
                       const int32_t* labels, cudaStream_t s);
void launch_prefill_advance(const State& st, int S, cudaStream_t s);
void launch_init_window(const State& st, uint32_t seed_lo, uint32_t seed_hi, cudaStream_t s);
void launch_export_tokens(const State& st, int32_t* out, cudaStream_t s);
// synthetic state for the threshold calibration: the first `live` images at cursor T/2, the rest finished
void launch_calib_state(const State& st, int live, cudaStream_t s);
void launch_prob_accept(const State& st, const AcceptArgs& a, cudaStream_t s);
void launch_commit(const State& st, const AcceptArgs& a, cudaStream_t s);
// smallest commit over the live slots of this round, from the accept flags (batch-synchronous progress)
void launch_sync_min(const State& st, const AcceptArgs& a, int32_t* m_sync, cudaStream_t s);
int accept_smem_bytes(int V);
// persistent form of launch_prob_accept for vocabularies up to 16384 (accept_persistent.cu)
bool accept_persistent_supported(const State& st);
void launch_accept_persistent(const State& st, const AcceptArgs& a, int n_sms, cudaStream_t s);
// streaming multiprocessors of the current device
int device_sm_count();
void launch_probs(const float* lc, const float* lu, int rows, int V, float cfg_scale, float temperature, int top_k,
                  float* p, cudaStream_t s);

// empty kernel launched like every other (timing aid, model_kernels.cu)
void launch_noop(cudaStream_t s);

// ---- distillation score (score_kernels.cu)
void launch_bikl_rows(const float* ls, const float* lt, int rows, int V, float* out, cudaStream_t s);
// terms of the inputs of one scoring chunk (slot tables of st; logits rows slot * W + i of both models)
void launch_bikl_slots(const State& st, int S, const float* ls, const float* lt, const int32_t* prefix_len,
                       float* pos, cudaStream_t s);
void launch_score_init(const State& st, const int32_t* tokens, const int32_t* labels, const int32_t* prefix_len,
                       float* pos, cudaStream_t s);
void launch_score_reduce(int B, int T, const int32_t* prefix_len, const float* pos, float* per_image, float* loss,
                         cudaStream_t s);

// ---- tcgen05 GEMM (gemm_tcgen05.cu)
// C[M,N] fp32 (+)= A[M,K] bf16 . W[N,K]^T bf16.  force_bn: 0 = choose the tile width from the shape.
// error_flag: device int set non-zero if a bounded pipeline wait gave up.  Returns 0, or a negative
// code with a message in err.
// m_cap (>= M, or 0): row capacity of the A and C buffers; lets one cached tensor map serve every M.
// w_constant: W is a model weight (never written while the stream runs), so its first tiles may be fetched before
// the preceding kernel has finished.  acc_wait_ns: 0, or a shorter limit of the epilogue's accumulator wait.
int gemm_tcgen05_run(const bf16* A, const bf16* W, float* C, int M, int N, int K, int accumulate, int force_bn,
                     int m_cap, int32_t* error_flag, cudaStream_t s, char* err, size_t errlen, int w_constant = 1,
                     unsigned int acc_wait_ns = 0);
int gemm_tcgen05_tile_n(int M, int N, int K);
// Cached TMA descriptor of a row-major bf16 matrix [rows, cols]: box = 64 columns x box_rows rows, 128-byte swizzle.
bool make_tensor_map_bf16(::CUtensorMap_st* map, const void* base, int rows, int cols, int box_rows);
// RMSNorm folded around a GEMM: A holds the bf16 copy of the unnormalised residual rows x, W has the norm's gain
// folded in, and the epilogue multiplies row m by rsqrt(sum(ssq[m][0 .. K/32)) / K + eps).  ssq null: no factor.
struct NormIn {
    const float* ssq;  // [M][K / 32] partial sums of squares of the fp32 rows
    float eps;
};
// act[M, F] bf16 = silu(gate) * up, from A[M,K] . W13i^T where W13i[2F, K] holds gate row f at 2f, up row f at 2f+1.
int gemm_tcgen05_swiglu(const bf16* A, const bf16* W13_interleaved, bf16* act, int M, int F2, int K, int m_cap,
                        const NormIn& nin, int32_t* error_flag, cudaStream_t s, char* err, size_t errlen);
// logits[M, N] fp32 = norm(x) . W^T with the norm folded as above.
int gemm_tcgen05_head(const bf16* A, const bf16* W, float* C, int M, int N, int K, int m_cap, const NormIn& nin,
                      int32_t* error_flag, cudaStream_t s, char* err, size_t errlen);
// Residual update h[M, N] fp32 += A[M,K] . W^T, which also leaves what the next folded norm needs: hb = bf16(h)
// and ssq_out[M][N / 32] = sums of squares of the new h over each 32-column chunk (fixed order, no atomics).
int gemm_tcgen05_addnorm(const bf16* A, const bf16* W, float* h, bf16* hb, float* ssq_out, int M, int N, int K,
                         int m_cap, int32_t* error_flag, cudaStream_t s, char* err, size_t errlen);
// QKV projection of the normed activations A[M, D] with the 2D RoPE and the paged KV write fused:
// q[M, D] bf16 rotated; rotated k and v stored at each row's (cache row, sequence index).
int gemm_tcgen05_qkv(const bf16* A, const bf16* Wqkv, bf16* q, const State& st, int S, int layer,
                     const float* rope_cs, const KvView& kv, int m_cap, const NormIn& nin, int32_t* error_flag,
                     cudaStream_t s, char* err, size_t errlen);

}  // namespace hbsjd
