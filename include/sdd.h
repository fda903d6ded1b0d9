/*
 * sdd.h — C ABI of the Speculative Diffusion Decoding (SpecDiff) round for NVIDIA B200 (sm_100a).
 *
 * One SpecDiff round (Algorithm 1 of "Speculative Diffusion Decoding", arXiv 2408.05636):
 *   draft   : a masked-diffusion drafter M_q fills gamma [MASK] slots appended to the context in
 *             T denoising evaluations (non-causal forward, soft-max over the vocabulary, draw);
 *   verify  : the autoregressive target M_p scores all gamma+1 positions in one causal forward;
 *   accept  : drafted token j is kept while u_j <= min(1, p_j(x_j)/q_j(x_j)); the first rejected
 *             position is redrawn from norm(max(0, p - q)); if none is rejected one more token
 *             is drawn from p_{gamma+1}.
 *
 * Conventions
 *   - Every function returns an int32 status: SDD_OK (0) or a negative SDD_E_* code.  Nothing
 *     here aborts, throws, traps the device or allocates device memory: the caller owns the
 *     weights, the prompt, the outputs and one workspace blob whose size the library reports.
 *     (The library owns only small host-side bookkeeping, including a few pinned host words.)
 *   - "device" pointers are CUDA device pointers valid on the current device; "host" pointers
 *     are ordinary host memory.  Pointers are borrowed for the lifetime of the sdd_ctx.
 *   - All work is enqueued on the caller's stream and is asynchronous; only sdd_sync_status
 *     blocks.  One sdd_ctx must be driven from one host thread at a time.
 *   - Both networks are GPT-2-shaped (learned token + position embeddings, pre-LayerNorm blocks
 *     with fused QKV, tanh-GELU MLP of width 4d, final LayerNorm, LM head tied to the token
 *     embedding).  The drafter has one extra embedding row, id == vocab, the [MASK] token, and
 *     uses no attention mask; the target is causal.
 *   - Randomness: Philox4x32-10 keyed by `seed`; counter = (v >> 2 | 0, slot j, round r,
 *     purpose << 24 | step k << 16 | sequence b); uniform = ((word >> 9) + 0.5) * 2^-23;
 *     categorical draws are Gumbel-max over the vocabulary (ties -> lowest id).
 */
#ifndef SDD_H_
#define SDD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  SDD_OK = 0,
  SDD_E_ARG = -1,        /* null pointer, non-positive size, unsupported option               */
  SDD_E_SHAPE = -2,      /* model shapes unsupported or inconsistent (vocab, d_model % n_head) */
  SDD_E_WORKSPACE = -3,  /* workspace too small or misaligned (needs 256-byte alignment)       */
  SDD_E_CTX_FULL = -4,   /* prompt + max_new + gamma exceeds a model's n_ctx                   */
  SDD_E_CUDA = -5,       /* a CUDA runtime / driver call failed (see sdd_last_cuda_error)      */
  SDD_E_TIMEOUT = -6,    /* a bounded device-side wait ran out; the device stays usable        */
  SDD_E_UNIMPL = -7,     /* option combination not implemented                                 */
  SDD_E_STATE = -8,      /* call order violated (e.g. verify before draft)                     */
  SDD_E_INDEX = -9       /* a token id outside [0, vocab) reached the device (prompt or draft ids):
                            it was replaced by a zero embedding / a rejected draft, never used as an
                            index; reported by sdd_sync_status                                     */
};

enum { SDD_FP32 = 0, SDD_BF16 = 1 };

/* One transformer.  `tensors` is a host array of `n_tensors` device pointers in this order:
 *   wte [vocab (+1 for the drafter), d], wpe [n_ctx, d],
 *   then for each layer: ln1_g[d] ln1_b[d] w_qkv[3d,d] b_qkv[3d] w_o[d,d] b_o[d]
 *                        ln2_g[d] ln2_b[d] w_fc1[4d,d] b_fc1[4d] w_fc2[d,4d] b_fc2[d],
 *   then lnf_g[d] lnf_b[d].                       (n_tensors = 2 + 12 * n_layer + 2)
 * Linear weights are [out_features, in_features] row-major (y = x W^T + b).  With dtype ==
 * SDD_BF16 the matrices (wte, wpe, w_*) are bf16 and the vectors (ln*, b_*) are fp32; with
 * SDD_FP32 everything is fp32.  All pointers must be 16-byte aligned.  The tensors are borrowed and must
 * not change while a context that uses them has work queued: kernels read weight tiles before they wait for
 * the work ahead of them in the stream. */
typedef struct {
  int32_t vocab, n_layer, d_model, n_head, n_ctx;
  int32_t causal; /* 1 = autoregressive target, 0 = masked-diffusion drafter */
  int32_t dtype;  /* SDD_FP32 or SDD_BF16 */
  const void* const* tensors;
  int32_t n_tensors;
} sdd_model;

typedef struct {
  int32_t gamma;   /* draft length, 1..256                                                     */
  int32_t T;       /* denoising evaluations per round, 1..255                                   */
  int32_t batch;   /* independent sequences, 1..65535                                           */
  int32_t max_new; /* tokens to generate per sequence; the last round's emission is truncated   */
  float temp_p;    /* target temperature; 0 = greedy                                            */
  float temp_q;    /* drafter temperature; 0 = greedy (temp_p and temp_q must both be 0 or > 0) */
  uint64_t seed;   /* Philox key                                                                */
  void* stream;    /* cudaStream_t, borrowed                                                    */
} sdd_params;

typedef struct sdd_ctx sdd_ctx;

/* Bytes of device workspace sdd_create needs for these models and parameters (host call). */
int32_t sdd_workspace_bytes(const sdd_model* target, const sdd_model* drafter, const sdd_params* params,
                            uint64_t* out_bytes);

/* Set up one generation (Section "Preliminaries": prefix x_{1:i} in, next n tokens out).
 *   prompt_ids : device int32 [batch, prompt_stride], row b holds prompt_len[b] ids in [0, vocab)
 *                (the host cannot see them: an id outside that range becomes a zero embedding row on
 *                the device and sdd_sync_status returns SDD_E_INDEX)
 *   prompt_len : host int32 [batch], each >= 1
 *   workspace  : device memory, 256-byte aligned, >= sdd_workspace_bytes(); zeroed by this call
 * Also enqueues the target's prefill of x_{0:c-2} into its KV cache.  *out receives the context
 * (free it with sdd_destroy).  Errors: SDD_E_ARG, SDD_E_SHAPE, SDD_E_WORKSPACE, SDD_E_CTX_FULL,
 * SDD_E_CUDA. */
int32_t sdd_create(const sdd_model* target, const sdd_model* drafter, const sdd_params* params,
                   const int32_t* prompt_ids, int32_t prompt_stride, const int32_t* prompt_len,
                   void* workspace, uint64_t workspace_bytes, sdd_ctx** out);

/* A new generation in the same context (the paper has the loop of rounds only; this is what a server does between
 * requests): same models, parameters, workspace, stream and captured graphs, new prompts.  Arguments as for
 * sdd_create (prompt_ids device int32 [batch][prompt_stride], prompt_len host int32 [batch]).  Synchronises the
 * stream first (rounds of the old generation still in flight finish), restarts the round counter -- and with it the
 * random streams, so the result equals that of a fresh context with the same seed --, reloads and prefills.  An
 * attached autoregressive drafter is prefilled again and sdd_sps_step is allowed again.  SDD_E_STATE inside a round,
 * SDD_E_CTX_FULL / SDD_E_ARG as for sdd_create. */
int32_t sdd_reset(sdd_ctx* ctx, const int32_t* prompt_ids, int32_t prompt_stride, const int32_t* prompt_len);

/* Drafting (Algorithm 1, the loop over the T diffusion steps and the draw of the draft from q^0):
 *   sdd_draft_begin : all gamma slots <- [MASK]
 *   sdd_draft_step  : one denoising evaluation k = T, T-1, ... : drafter forward over
 *                     context ∘ slots, LM head on the slot rows, then each still-masked slot is
 *                     revealed with probability 1/k by a Gumbel-max draw from softmax(l / temp_q);
 *                     the revealing row's logits and log q(x) are stored for the acceptance test
 *   sdd_draft       : begin + T steps
 * SDD_E_STATE if more than T steps are requested in one round. */
int32_t sdd_draft_begin(sdd_ctx* ctx);
int32_t sdd_draft_step(sdd_ctx* ctx);
int32_t sdd_draft(sdd_ctx* ctx);

/* Verification and acceptance (Algorithm 1 from the parallel evaluation of M_p to its return statement): one causal,
 * KV-cached target forward over [last context token, draft_1..draft_gamma], the acceptance test,
 * the extra token, and the commit of n+1 tokens to every sequence's context.  Requires a finished
 * draft (SDD_E_STATE otherwise).  If non-null, out_ids (device int32 [batch, gamma+1]) receives
 * the tokens emitted this round (-1 padded) and n_out (device int32 [batch]) their count per
 * sequence (0 for a sequence that already has max_new tokens).  Both may also point to page-locked host memory
 * that the device can address: the commit kernel then writes them over the bus, and they are complete for round r
 * as soon as sdd_progress reports r + 1 rounds, without a stream synchronisation. */
int32_t sdd_verify_accept(sdd_ctx* ctx, int32_t* out_ids, int32_t* n_out);

/* One whole round = sdd_draft + sdd_verify_accept. */
int32_t sdd_step(sdd_ctx* ctx, int32_t* out_ids, int32_t* n_out);

/* Plain autoregressive decoding of the target, one token per call: the "standard generation" that the paper's
 * speed-ups are quoted against (Table 1, row "Autoregressive"), expressed as a round with an empty draft (gamma = 0:
 * nothing to test, the emitted token is the draw from p).  May be mixed freely with sdd_step between rounds; the
 * Philox round index advances by one per call and the draw uses the bonus stream at slot 0.
 * out_ids: device int32 [batch] (one token per sequence, -1 if the sequence is complete), n_out: device int32 [batch];
 * either may be null. */
int32_t sdd_ar_step(sdd_ctx* ctx, int32_t* out_ids, int32_t* n_out);

/* Sequence initialisation (Section "Sequence initialization"; Table "walltime-metrics-prefix" samples the first 100
 * tokens this way): standard speculative decoding with an AUTOREGRESSIVE drafter for the first tokens of a
 * generation, SpecDiff rounds afterwards.  One such round is gamma_sps sequential evaluations of the drafter
 * (Section "Preliminaries and Settings", paragraph "Speculative decoding": x_{i+j} ~ q_{i+j}(. | x_{1:i+j-1}), every
 * q row stored) followed by the same verification, acceptance, extra-token and commit kernels as sdd_step.
 *
 * sdd_sps_workspace_bytes: bytes of the drafter's KV cache (+ a few ints) for params->batch sequences.
 * sdd_sps_attach: ar_drafter is a causal model (sdd_model, causal = 1) with the target's vocabulary and dtype and
 *   d_model <= the target's (it runs in the context's activation buffers); its weights stay owned by the caller and
 *   must outlive the context.  workspace: device memory, 256-byte aligned, owned by the caller until sdd_destroy.
 *   Must be called right after sdd_create (before any round: SDD_E_STATE otherwise); every prompt needs at least two
 *   tokens (SDD_E_ARG); the drafter's position table must cover prompt + max_new + gamma (SDD_E_CTX_FULL).  Enqueues
 *   the prefill of the drafter's cache on the context's stream.
 * sdd_sps_step: one speculative-decoding round; 1 <= gamma_sps <= params.gamma (SDD_E_ARG).  out_ids is device int32
 *   [batch][gamma_sps + 1] (-1 padded), n_out device int32 [batch]; either may be null.  The Philox round index is
 *   shared with the other rounds; the draft draw of slot j uses the same stream as a SpecDiff round's slot j.
 *   Allowed only while every round so far was a speculative-decoding round (the drafter's cache has no gaps then);
 *   after the first sdd_step / sdd_draft_begin / sdd_ar_step it returns SDD_E_STATE. */
int32_t sdd_sps_workspace_bytes(const sdd_model* ar_drafter, const sdd_params* params, uint64_t* out_bytes);
int32_t sdd_sps_attach(sdd_ctx* ctx, const sdd_model* ar_drafter, void* workspace, uint64_t workspace_bytes);
int32_t sdd_sps_step(sdd_ctx* ctx, int32_t gamma_sps, int32_t* out_ids, int32_t* n_out);

/* Non-blocking progress read (host): rounds whose commit has been seen so far, and the smallest
 * number of generated tokens over the batch at that point.  Either pointer may be null. */
int32_t sdd_progress(sdd_ctx* ctx, uint64_t* rounds_done, int32_t* min_emitted);

/* Stand-alone acceptance on given logits (the acceptance rule of Section "Preliminaries" and
 * Algorithm 1's last block, without the networks).  All pointers are device pointers.
 *   logits_p  fp32 [rows, gamma+1, V]   target logits, row j scores the token after draft[0:j]
 *   logits_q  fp32 [rows, gamma, V]     drafter logits each draft token was drawn from
 *   draft_ids int32 [rows, gamma]
 *   n_accept  int32 [rows]              out: number of accepted draft tokens
 *   out_ids   int32 [rows, gamma+1]     out: accepted tokens, then the extra token; rest = -1
 *   accept_prob fp32 [rows, gamma]      out: min(1, p/q) of every row (also past the rejection)
 *   scratch   device, >= sdd_accept_scratch_bytes(rows, gamma, V) bytes, 16-byte aligned
 * logits_p and logits_q must be 16-byte aligned.  Row b uses Philox sequence index b and round
 * index `round`, of which the low 32 bits are used (the Philox counter word that carries the round
 * is 32 bits wide; the rounds of a context are counted in 32 bits too).  rows <= 65535,
 * gamma <= 256, temp_p and temp_q both 0 (greedy) or both > 0.  A draft id outside [0, V) is never
 * used as an index: that sequence gets n_accept = -1 and out_ids all -1. */
uint64_t sdd_accept_scratch_bytes(int32_t rows, int32_t gamma, int32_t V);
int32_t sdd_accept_logits(const float* logits_p, const float* logits_q, const int32_t* draft_ids,
                          int32_t rows, int32_t gamma, int32_t V, float temp_p, float temp_q,
                          uint64_t seed, uint64_t round, int32_t* n_accept, int32_t* out_ids,
                          float* accept_prob, void* scratch, void* stream);

/* The same acceptance step for callers that cannot allocate device memory: code that runs where
 * cudaMalloc is off limits (a host whose memory pool was sized and handed out up front, a
 * real-time loop that must not enter the allocator, a plugin that is given its tensors and
 * nothing else) still has to place the per-chunk statistics somewhere, so this entry point keeps
 * them in a fixed array of SDD_ACCEPT_STATIC_SCRATCH_BYTES inside the library's device image.
 * (This call is a convenience of the library; the paper has no counterpart.)
 *   - Arguments and results are those of sdd_accept_logits, without `scratch`.
 *   - Sizes with rows * (2 gamma + 1) * ceil((V + 3) / 8192) * 8 bytes above the fixed size are
 *     refused with SDD_E_WORKSPACE; use sdd_accept_logits with your own scratch for those.
 *   - Every GPU that loads the library holds the array until the process exits.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current, as for every call here); make that first call before any stream capture.
 *   - All calls share the one array: two calls whose kernels may overlap on the GPU (different
 *     streams, or different host threads) race on it.  Calls on one stream are safe.  The array
 *     keeps the previous call's contents; nothing in it needs clearing, because each call writes
 *     every entry it later reads.
 *   - It calls no allocation routine of CUDA or of any other library. */
#define SDD_ACCEPT_STATIC_SCRATCH_BYTES (2u << 20)
int32_t sdd_accept_logits_static(const float* logits_p, const float* logits_q, const int32_t* draft_ids,
                                 int32_t rows, int32_t gamma, int32_t V, float temp_p, float temp_q,
                                 uint64_t seed, uint64_t round, int32_t* n_accept, int32_t* out_ids,
                                 float* accept_prob, void* stream);

/* Diagnostic: the library's bf16 GEMM on its own,  C[M, N] = A[M, K] W[N, K]^T  with fp32 accumulation
 * (the contraction used for the QKV / O / MLP / LM-head products of both networks' forwards).
 *   A   device bf16, dense [a_rows_capacity, K] of which the first M rows are used
 *   W   device bf16 [N, K];  bias device fp32 [N] or null
 *   epilogue 0: out bf16 = acc + bias; 1: out bf16 = gelu_tanh(acc + bias);
 *            2: out fp32 += acc + bias; 3: out fp32 = acc + bias       (out row stride ldc >= N)
 *   n_tile   0 = let the library choose, else 32 / 64 / 128 / 256 (only for M > 64)
 *   use_tensor_cores 1 = tcgen05 kernel, 0 = CUDA-core kernel
 *   status_word device int32 (may be null): set to 1 if a bounded device-side wait expired
 *   A_lo (may be null) second half of a hi/lo activation pair, same shape as A: the product uses A + A_lo
 *        (how the target's MLP and LM head carry their activations to about 16 significant bits)
 *   out_lo (may be null; epilogues 0 and 1) receives bf16(x - bf16(x)) next to out = bf16(x)
 * K must be a multiple of 8; A, A_lo and W 16-byte aligned.  W must be complete in memory when the call is made (not
 * the output of work still running on `stream`): like the weights of a model it is fetched before the kernel waits
 * for the work ahead of it in the stream. */
int32_t sdd_debug_gemm_bf16(const void* A, int64_t a_rows_capacity, const void* W, const float* bias, int32_t M,
                            int32_t N, int32_t K, int32_t epilogue, void* out, int32_t ldc, int32_t n_tile,
                            int32_t use_tensor_cores, int32_t* status_word, void* stream, const void* A_lo,
                            void* out_lo);

/* Diagnostic: the library's bf16 tensor-core attention on its own (d_head = 64), as used inside both
 * networks' blocks: out = softmax(Q K^T / 8 [+ mask]) V per head.
 *   q   device bf16 [q_rows_total, q_ld]; head h occupies columns q_col0 + 64 h .. ; sequence b owns rows
 *       b * q_rows_per_seq ..
 *   k   device bf16 [k_rows_total, k_ld], heads from column k_col0, sequence b owns rows b * k_rows_per_seq ..
 *   vt  device bf16 [batch * 64 n_head, vt_ld]: V transposed, row b * d + feature, column = key position
 *       (entries past the valid keys must be finite)
 *   out device bf16 [batch * q_rows_per_seq, ld_out]
 *   mode 0: no mask, rows and keys 0 .. ctx_len[b] + gamma - 1 (the drafter);
 *        1: row i is position ctx_len[b] - 1 + i and sees keys 0 .. that position (target verification);
 *        2: row i is position i, valid while i < ctx_len[b] - 1 (target prefill).
 * q_ld, k_ld, vt_ld, ld_out multiples of 8; all pointers 16-byte aligned. */
int32_t sdd_debug_attention_bf16(const void* q, int64_t q_rows_total, int32_t q_ld, int32_t q_col0, const void* k,
                                 int64_t k_rows_total, int32_t k_ld, int32_t k_col0, int32_t k_rows_per_seq,
                                 const void* vt, int32_t vt_ld, void* out, int32_t ld_out, const int32_t* ctx_len,
                                 int32_t batch, int32_t n_head, int32_t gamma, int32_t mode, int32_t q_rows_per_seq,
                                 int32_t* status_word, void* stream);

/* Diagnostic: one CTA with the tensor-core kernels' role layout (copy producer, MMA issuer, epilogue warps, TMEM
 * allocation) whose consumer waits on a barrier that nothing arrives on, with the kernels' own bounded wait and a
 * limit of limit_cycles SM clocks (1 .. 2e9).  The wait runs out, the CTA raises its abort flag and *status_word =
 * 1, every role leaves its loop, TMEM is freed and the kernel returns: the path a stuck copy or MMA would take in
 * the GEMM and attention kernels, exercised without a fault.  status_word: device int32, must be 0 before the call. */
int32_t sdd_debug_wait_timeout(int64_t limit_cycles, int32_t* status_word, void* stream);

/* Read-only device views into the workspace, for inspection and tests. */
enum {
  SDD_TAP_TOKENS = 0,      /* int32 [batch, tok_stride] context ids (prompt + emitted);
                              tok_stride = min(target.n_ctx, drafter.n_ctx)                     */
  SDD_TAP_CTX_LEN = 1,     /* int32 [batch]                                                     */
  SDD_TAP_DRAFT_IDS = 2,   /* int32 [batch, gamma]      slot ids (vocab = still [MASK])         */
  SDD_TAP_STEP_LOGITS = 3, /* fp32  [batch, gamma, V]   drafter logits of the latest evaluation */
  SDD_TAP_Q_LOGITS = 4,    /* fp32  [batch, gamma, V]   stored rows l / temp_q (raw l if greedy)*/
  SDD_TAP_LOGQ = 5,        /* fp32  [batch, gamma]      log q_j(x_j)                            */
  SDD_TAP_REVEAL_STEP = 6, /* int32 [batch, gamma]      k at which slot j was revealed          */
  SDD_TAP_LOGITS_P = 7,    /* fp32  [batch, gamma+1, V] target logits                           */
  SDD_TAP_ACCEPT_PROB = 8, /* fp32  [batch, gamma]      min(1, p/q)                             */
  SDD_TAP_N_ACCEPT = 9,    /* int32 [batch]                                                     */
  SDD_TAP_EXTRA_TOKEN = 10,/* int32 [batch]                                                     */
  SDD_TAP_N_EMITTED = 11,  /* int32 [batch]             tokens generated so far                 */
  SDD_TAP_STATUS = 12,     /* int32 [1]                 device status word (0 = ok)             */
  SDD_TAP_EVALS = 13       /* int32 [2]                 drafter evaluations of this generation that
                              ran / that were skipped because the step before revealed nothing  */
};
int32_t sdd_tap(sdd_ctx* ctx, int32_t what, const void** dev_ptr, uint64_t* bytes);

/* Host-side counters: rounds enqueued, kernels launched so far by this context. */
int32_t sdd_counters(sdd_ctx* ctx, uint64_t* rounds, uint64_t* kernel_launches);

/* Optional per-launch timing, for measurement only (it adds two CUDA events around every kernel
 * launch, so it is not meant to be left on).  sdd_profile_begin starts collecting; sdd_profile_end
 * synchronises the stream and returns, per kernel category, the summed device time in milliseconds
 * and the number of launches (arrays of n_categories >= SDD_PROF_COUNT entries).  The event pairs are
 * recorded inside the round's graph; the cost of an empty pair, measured in the same graph, is subtracted. */
enum {
  SDD_PROF_GEMM_DRAFTER = 0, SDD_PROF_GEMM_TARGET = 1, SDD_PROF_HEAD_DRAFTER = 2, SDD_PROF_HEAD_TARGET = 3,
  SDD_PROF_ATTN_DRAFTER = 4, SDD_PROF_ATTN_TARGET = 5, SDD_PROF_LAYERNORM = 6, SDD_PROF_GLUE = 7,
  SDD_PROF_SAMPLE = 8, SDD_PROF_ROW_STATS = 9, SDD_PROF_ACCEPT = 10, SDD_PROF_COMMIT = 11, SDD_PROF_COUNT = 12
};
int32_t sdd_profile_begin(sdd_ctx* ctx);
int32_t sdd_profile_end(sdd_ctx* ctx, double* ms_per_category, uint64_t* launches_per_category,
                        int32_t n_categories);

/* Synchronise the stream and return the device status word as an SDD_E_* code. */
int32_t sdd_sync_status(sdd_ctx* ctx);

void sdd_destroy(sdd_ctx* ctx);
const char* sdd_strerror(int32_t status);
/* Text of the last CUDA error seen by this thread's calls into the library ("" if none). */
const char* sdd_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SDD_H_ */
