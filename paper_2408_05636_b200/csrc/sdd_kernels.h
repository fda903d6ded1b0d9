// Internal launcher interface between the round scheduler (sdd_api.cu) and the kernels.
#pragma once

#include "sdd_common.cuh"

namespace sdd {

// ---- device-resident round state (head of the workspace) ------------------------------------
struct RoundState {
  int status;          // DEV_OK or the first device-side error
  uint32_t round;      // rounds committed so far == Philox round index of the round in flight
  uint32_t revealed;   // slots revealed by the denoising step in flight (all sequences)
  uint32_t ticket;     // CTAs of that step's sampling kernel that have finished
  int skip_forward;    // 1: the last step revealed nothing, so the next drafter evaluation would reproduce the
                       //    logits it already has ("cache" strategy): its kernels return at once
  int evals_run;       // drafter evaluations of this generation that ran ...
  int evals_skipped;   // ... and that were skipped on skip_forward (counted by the sampling kernel's last CTA)
  int pad[1];
};

// How a target forward maps its rows to sequence positions.
//   VERIFY : row j of sequence b is position ctx_len[b] - 1 + j, j = 0..gamma          (all rows valid)
//   PREFILL: row j of sequence b is position j, valid while j < ctx_len[b] - 1
enum TargetMode : int { TARGET_VERIFY = 0, TARGET_PREFILL = 1 };

// GEMM epilogues:  C = A W^T (+ bias)
enum Epilogue : int {
  EPI_STORE = 0,      // out (activation type) = acc + bias
  EPI_GELU = 1,       // out (activation type) = gelu_tanh(acc + bias)
  EPI_RESIDUAL = 2,   // resid (fp32) += acc + bias
  EPI_STORE_F32 = 3,  // out (fp32) = acc            (LM head; ldc may differ from N)
  EPI_QKV = 4         // fused-QKV projection of the tensor-core path: Q (and the drafter's K) to `out`,
                      // the target's K to its cache, V transposed ([feature][position]) -- see QkvDst
};

// Destinations of the EPI_QKV epilogue.  Token row tr belongs to sequence b = tr / rows_per_seq at local
// index i = tr % rows_per_seq; its position is i (mode 0 drafter, mode 2 prefill, valid while i < c - 1)
// or c - 1 + i (mode 1 verify), with c = ctx_len[b].
struct QkvDst {
  __nv_bfloat16* k_dst;   // null: K is stored to `out` next to Q; else K cache [B][k_seq_rows][d]
  __nv_bfloat16* vt_dst;  // V^T [B][d][vt_ld]
  const int* ctx_len;
  int rows_per_seq, mode, d, k_seq_rows, vt_ld;
};

// Soft-max statistics of the logit rows computed in the epilogue of the tensor-core LM head (persistent kernels), so
// that no kernel has to read the (gamma + 1) x V logits again for them: per (token row, slice of the vocabulary) one
// pair (max z, sum exp(z - max)) with z = logit * inv_tau -- greedy (inv_tau == 0): (max logit, index of the first
// maximum as int bits) -- at partial[row * chunks + slice], the layout the acceptance kernel merges.
struct HeadStats {
  float inv_tau;
  float2* partial;        // null: no statistics
  int chunks_capacity;    // pairs per row that `partial` has room for
};
int head_stats_chunks_max(int V);   // pairs per row the fused statistics may need for a vocabulary of V

// Every kernel of a drafter evaluation takes `skip` (may be null): when *skip != 0 the kernel returns at once.

// ---- vocabulary kernels (sdd_sample.cu) -----------------------------------------------------
int stats_chunks_for(int V);
cudaError_t launch_row_stats(const float* a, long long rows_a, const float* b, long long rows_b, int V, float inv_tau_a,
                             float inv_tau_b, float2* partial, cudaStream_t st);
// lseq [batch, gamma] receives the log-sum-exp of every stored q row (the acceptance step's residual draw reads it)
cudaError_t launch_unmask_sample(const float* step_logits, int* slot_ids, float* q_logits, float* logq, float* lseq,
                                 int* reveal_step, int batch, int gamma, int V, int k, float inv_tau_q, PhiloxKey key,
                                 RoundState* rs, int cache_skip, cudaStream_t st);
// round pipeline: logq_in / lseq_in from the draws, partial_q null; stand-alone: logq_in / lseq_in null, partial_q given
// chunks_p / chunks_q: pairs per row in partial_p / partial_q
cudaError_t launch_accept(const float* logits_p, const float* q_rows, const int* draft_ids, const float* logq_in,
                          const float* lseq_in, const float2* partial_p, int chunks_p, const float2* partial_q, int chunks_q,
                          int rows, int gamma, int V,
                          float inv_tau_p, float inv_tau_q_rows, PhiloxKey key, uint32_t rnd, RoundState* rs, float* accept_prob,
                          int* n_accept, int* extra_token, int* out_ids, cudaStream_t st);
cudaError_t launch_commit(int* tokens, int tok_stride, int* ctx_len, int* n_emitted, const int* slot_ids,
                          const int* n_accept, const int* extra_token, int batch, int gamma, int max_new, RoundState* rs,
                          int* out_ids, int* n_out, volatile int* host_mirror, cudaStream_t st);
// draw of slot j from the last of the rows_per_seq logit rows per sequence (autoregressive drafter)
cudaError_t launch_ar_sample(const float* logits, int rows_per_seq, int* slot_ids, float* q_logits, float* logq, float* lseq,
                             int* reveal_step, int batch, int gamma, int j, int V, float inv_tau_q, PhiloxKey key,
                             RoundState* rs, cudaStream_t st);
cudaError_t launch_reset_slots(int* slot_ids, int* reveal_step, int n, int mask_id, RoundState* rs, cudaStream_t st);

// ---- glue (sdd_glue.cu) ---------------------------------------------------------------------
template <typename T>
cudaError_t launch_embed_drafter(const T* wte, const T* wpe, const int* tokens, int tok_stride, const int* ctx_len,
                                 const int* slot_ids, int batch, int gamma, int L_cap, int d, float* h, cudaStream_t st,
                                 const int* skip = nullptr, const float* ln_g = nullptr, const float* ln_b = nullptr,
                                 T* xn = nullptr,    // xn != null: also xn = LayerNorm(h; ln_g, ln_b), the first block's
                                 int vocab = 0x7fffffff, int* status = nullptr);
// Token ids index the embedding tables, so every embedding kernel checks them: an id outside [0, vocab) (the drafter
// also takes vocab, its [MASK] row) gives a zero embedding row and raises DEV_BAD_TOKEN in *status (if non-null).
template <typename T>
cudaError_t launch_embed_target(const T* wte, const T* wpe, const int* tokens, int tok_stride, const int* ctx_len,
                                const int* slot_ids, int batch, int gamma, int rows_per_seq, int mode, int d, float* h,
                                cudaStream_t st, int vocab = 0x7fffffff, int* status = nullptr);
// rows of an autoregressive drafter's evaluation: positions ctx_len[b] + off - 1 + i; writes eff_len[b] = ctx_len[b] + off
template <typename T>
cudaError_t launch_embed_ar(const T* wte, const T* wpe, const int* tokens, int tok_stride, const int* ctx_len,
                            const int* slot_ids, int batch, int gamma, int rows_per_seq, int off, int d, float* h,
                            int* eff_len, cudaStream_t st, int vocab = 0x7fffffff, int* status = nullptr);
// LayerNorm of `rows` rows of h (fp32, row stride d) into out (activation type); out_lo (optional) receives the
// rounding remainder y - out so that (out, out_lo) carries y to about 16 significant bits
template <typename T>
cudaError_t launch_layernorm(const float* h, const float* g, const float* b, T* out, long long rows, int d, cudaStream_t st,
                             T* out_lo = nullptr, const int* skip = nullptr);
// final LayerNorm of the gamma slot rows of every sequence: out[b*gamma + j] = LN(h[b*L_cap + ctx_len[b] + j])
template <typename T>
cudaError_t launch_layernorm_slots(const float* h, const float* g, const float* b, T* out, const int* ctx_len, int batch,
                                   int gamma, int L_cap, int d, cudaStream_t st, const int* skip = nullptr);
// compact copies of the gamma slot rows of every sequence: att_s / h_s [batch * gamma, d]
template <typename T>
cudaError_t launch_gather_slots(const T* att, const float* h, const int* ctx_len, int batch, int gamma, int L_cap, int d,
                                T* att_s, float* h_s, cudaStream_t st, const int* skip = nullptr);
// copy the K and V thirds of qkv rows into the cache: cache[b][pos][0|1][d]
template <typename T>
cudaError_t launch_kv_append(const T* qkv, T* cache, const int* ctx_len, int batch, int rows_per_seq, int mode, int n_ctx,
                             int d, cudaStream_t st);

// ---- GEMM (sdd_gemm_simt.cu, sdd_gemm_tc.cu) ------------------------------------------------
// C[M, N] = A[M, K] * W[N, K]^T; A row stride lda, W row stride K, out row stride ldc.
template <typename T>
cudaError_t launch_gemm_simt(const T* A, int lda, const T* W, const float* bias, int M, int N, int K, int epi, void* out,
                             int ldc, cudaStream_t st, const int* skip = nullptr);

// bf16 tensor-core GEMM (tcgen05 / TMEM / TMA).  A is a dense [a_cap, K] buffer of which M rows are used;
// bn_hint selects the N tile (0 = choose); a bounded wait that expires sets *status = DEV_TIMEOUT.
// A_lo (optional): second half of a hi/lo activation pair, same shape as A; the product uses A + A_lo.
// out_lo (optional, bf16 epilogues): receives bf16(x - bf16(x)) next to out = bf16(x).
cudaError_t launch_gemm_tc(const __nv_bfloat16* A, long long a_cap, const __nv_bfloat16* W, const float* bias, int M, int N,
                           int K, int epi, void* out, int ldc, int bn_hint, int* status, cudaStream_t st,
                           const QkvDst* qkv = nullptr, const __nv_bfloat16* A_lo = nullptr, void* out_lo = nullptr,
                           const int* skip = nullptr, const HeadStats* stats = nullptr, int* stats_chunks = nullptr);
// stats (EPI_STORE_F32 only): where the launch runs on a persistent kernel the epilogue also writes the rows' soft-max
// statistics and *stats_chunks receives the number of pairs per row (0: not written, the caller runs row_stats)

// one CTA whose bounded waits run out after limit_cycles (see sdd_debug_wait_timeout)
cudaError_t launch_wait_timeout_probe(long long limit_cycles, int* status, cudaStream_t st);

// one-time set-up of the tensor-core kernels (dynamic shared-memory limits); also done lazily on first launch
cudaError_t tc_prepare_gemm();
cudaError_t tc_prepare_attn();

// bf16 tensor-core attention, d_head = 64 (sdd_attn_tc.cu).  q / k are row-major tensors with the heads side by
// side starting at column q_col0 / k_col0; vt is V transposed: [batch * d rows, vt_ld positions].
// mode 0: drafter (no mask, ctx_len[b] + gamma rows and keys); 1: target verify; 2: target prefill.
cudaError_t launch_attn_tc(const __nv_bfloat16* q, long long q_rows_total, int q_ld, int q_col0, const __nv_bfloat16* k,
                           long long k_rows_total, int k_ld, int k_col0, int k_rows_per_seq, const __nv_bfloat16* vt,
                           int vt_ld, __nv_bfloat16* out, int ld_out, const int* ctx_len, int batch, int n_head, int d,
                           int gamma, int mode, int q_rows_per_seq, int* status, cudaStream_t st,
                           const int* skip = nullptr);

// ---- attention (sdd_attn.cu) ----------------------------------------------------------------
// drafter: every row of a sequence attends to rows 0 .. ctx_len[b] + gamma - 1 of the same sequence
template <typename T>
cudaError_t launch_attn_bidir(const T* qkv, T* out, const int* ctx_len, int batch, int gamma, int L_cap, int n_head,
                              int d_head, cudaStream_t st, const int* skip = nullptr);
// target: row j of sequence b (position p, see TargetMode) attends to cache positions 0 .. p
template <typename T>
cudaError_t launch_attn_cached(const T* qkv, const T* cache, T* out, const int* ctx_len, int batch, int rows_per_seq,
                               int mode, int n_ctx, int n_head, int d_head, cudaStream_t st);

}  // namespace sdd
