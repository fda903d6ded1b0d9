// C ABI of the SpecDiff round: argument checking, workspace layout, and the host-side schedule
// that enqueues the kernels of Algorithm 1 on the caller's stream.  See include/sdd.h.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>
#include <tuple>
#include <type_traits>
#include <vector>

#include "sdd_kernels.h"

namespace sdd {

static thread_local char g_cuda_err[512] = "";

bool pdl_enabled() {
  static const bool on = [] {
    const char* e = getenv("SDD_PDL");
    return e == nullptr || atoi(e) != 0;
  }();
  return on;
}

static int cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
  return SDD_E_CUDA;
}
#define SDD_CUDA(expr)                                   \
  do {                                                   \
    cudaError_t e__ = (expr);                            \
    if (e__ != cudaSuccess) return cuda_fail(e__, #expr); \
  } while (0)
#define SDD_TRY(expr)               \
  do {                              \
    int s__ = (expr);               \
    if (s__ != SDD_OK) return s__;  \
  } while (0)

constexpr int ROW_TILE = 128;  // drafter rows per sequence are padded to a multiple of this

// kernel categories of the optional per-launch timing (sdd_profile_*)
enum Cat : int { CAT_GEMM_Q = 0, CAT_GEMM_P, CAT_HEAD_Q, CAT_HEAD_P, CAT_ATTN_Q, CAT_ATTN_P, CAT_LAYERNORM, CAT_GLUE,
                 CAT_SAMPLE, CAT_STATS, CAT_ACCEPT, CAT_COMMIT, CAT_COUNT };

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- one model's tensors, typed -------------------------------------------------------------
struct Layer {
  const float *ln1_g, *ln1_b, *b_qkv, *b_o, *ln2_g, *ln2_b, *b_fc1, *b_fc2;
  const void *w_qkv, *w_o, *w_fc1, *w_fc2;
};
struct Net {
  int vocab, n_layer, d, n_head, d_head, n_ctx, causal, dtype;
  const void *wte, *wpe;
  const float *lnf_g, *lnf_b;
  std::vector<Layer> layers;
};

static int parse_model(const sdd_model* m, int want_causal, Net* net) {
  if (m == nullptr || m->tensors == nullptr) return SDD_E_ARG;
  if (m->vocab < 2 || m->n_layer < 1 || m->d_model < 32 || m->n_head < 1 || m->n_ctx < 2) return SDD_E_SHAPE;
  if (m->d_model % m->n_head != 0 || m->d_model > 2048 || m->d_model % 8 != 0) return SDD_E_SHAPE;
  const int dh = m->d_model / m->n_head;
  if (dh != 32 && dh != 64) return SDD_E_SHAPE;
  if (m->causal != want_causal) return SDD_E_ARG;
  if (m->dtype != SDD_FP32 && m->dtype != SDD_BF16) return SDD_E_ARG;
  if (m->n_tensors != 2 + 12 * m->n_layer + 2) return SDD_E_SHAPE;
  for (int i = 0; i < m->n_tensors; ++i) {
    if (m->tensors[i] == nullptr) return SDD_E_ARG;
    if ((reinterpret_cast<uintptr_t>(m->tensors[i]) & 15u) != 0) return SDD_E_ARG;
  }
  net->vocab = m->vocab; net->n_layer = m->n_layer; net->d = m->d_model; net->n_head = m->n_head;
  net->d_head = dh; net->n_ctx = m->n_ctx; net->causal = m->causal; net->dtype = m->dtype;
  const void* const* t = m->tensors;
  net->wte = t[0]; net->wpe = t[1];
  net->layers.resize(m->n_layer);
  for (int l = 0; l < m->n_layer; ++l) {
    const void* const* p = t + 2 + 12 * l;
    Layer& L = net->layers[l];
    L.ln1_g = (const float*)p[0]; L.ln1_b = (const float*)p[1]; L.w_qkv = p[2]; L.b_qkv = (const float*)p[3];
    L.w_o = p[4]; L.b_o = (const float*)p[5]; L.ln2_g = (const float*)p[6]; L.ln2_b = (const float*)p[7];
    L.w_fc1 = p[8]; L.b_fc1 = (const float*)p[9]; L.w_fc2 = p[10]; L.b_fc2 = (const float*)p[11];
  }
  net->lnf_g = (const float*)t[2 + 12 * m->n_layer];
  net->lnf_b = (const float*)t[3 + 12 * m->n_layer];
  return SDD_OK;
}

// ---- workspace ------------------------------------------------------------------------------
struct Buffers {
  RoundState* rs;
  int *tokens, *ctx_len, *n_emitted, *slot_ids, *reveal_step, *n_accept, *extra_token;
  float *logq, *lse_q, *accept_prob;   // lse_q: log-sum-exp of every stored q row
  float *step_logits, *q_logits, *logits_p;
  float2* partial_p;
  float* h;                    // residual stream, fp32
  void *xn, *qkv, *att, *mlp, *xf;  // activations in the model dtype
  void *xn_lo, *mlp_lo, *xf_lo;  // rounding remainders of xn / mlp / xf (hi/lo pairs of the target's MLP and LM head)
  float* h_s;                  // residual stream of the gamma slot rows [batch * gamma, d_q] (last drafter block)
  void* vt;                    // drafter V transposed [batch][d_q][lcap_max] (tensor-core path)
  void* kv;                    // target KV cache [layer][batch][n_ctx][2][d]
};

struct Dims {
  int batch, gamma, T, max_new, V, tok_stride, chunks;
  int chunks_cap;              // pairs per row that partial_p has room for (the LM head's fused statistics need more than row_stats)
  int lcap_max;                // padded rows per sequence of the largest drafter forward
  long long rows_q, rows_p;    // largest row counts of a drafter / target forward
  int max_prompt;
  size_t esize;                // bytes of an activation element
};

static size_t carve(const Dims& D, const Net& P, const Net& Q, uint8_t* base, Buffers* B) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> uint8_t* {
    uint8_t* p = base ? base + off : nullptr;
    off = align_up(off + bytes, 256);
    return p;
  };
  const size_t Bn = D.batch, G = D.gamma, V = D.V;
  Buffers b;
  b.rs = (RoundState*)take(sizeof(RoundState));
  b.tokens = (int*)take(Bn * D.tok_stride * 4);
  b.ctx_len = (int*)take(Bn * 4);
  b.n_emitted = (int*)take(Bn * 4);
  b.slot_ids = (int*)take(Bn * G * 4);
  b.reveal_step = (int*)take(Bn * G * 4);
  b.n_accept = (int*)take(Bn * 4);
  b.extra_token = (int*)take(Bn * 4);
  b.logq = (float*)take(Bn * G * 4);
  b.lse_q = (float*)take(Bn * G * 4);
  b.accept_prob = (float*)take(Bn * G * 4);
  b.step_logits = (float*)take(Bn * G * V * 4);
  b.q_logits = (float*)take(Bn * G * V * 4);
  b.logits_p = (float*)take(Bn * (G + 1) * V * 4);
  b.partial_p = (float2*)take(Bn * (G + 1) * D.chunks_cap * sizeof(float2));
  const size_t rq = (size_t)D.rows_q, rp = (size_t)D.rows_p;
  auto mx = [](size_t a, size_t c) { return a > c ? a : c; };
  b.h = (float*)take(mx(rq * Q.d, rp * P.d) * 4);
  b.xn = take(mx(rq * Q.d, rp * P.d) * D.esize);
  b.qkv = take(mx(rq * Q.d, rp * P.d) * 3 * D.esize);
  b.att = take(mx(rq * Q.d, rp * P.d) * D.esize);
  b.mlp = take(mx(rq * Q.d, rp * P.d) * 4 * D.esize);
  b.xf = take(Bn * (G + 1) * mx(Q.d, P.d) * D.esize);
  b.vt = take(Bn * (size_t)Q.d * D.lcap_max * D.esize);
  // same capacities as their hi halves, so that one tensor-map extent describes both
  b.xn_lo = take(mx(rq * Q.d, rp * P.d) * D.esize);
  b.mlp_lo = take(mx(rq * Q.d, rp * P.d) * 4 * D.esize);
  b.xf_lo = take(Bn * (G + 1) * mx(Q.d, P.d) * D.esize);
  b.h_s = (float*)take(Bn * G * Q.d * 4);
  b.kv = take((size_t)P.n_layer * Bn * P.n_ctx * 2 * P.d * D.esize);
  if (B) *B = b;
  return off;
}

}  // namespace sdd

using namespace sdd;

struct sdd_ctx {
  Net P, Q;
  Dims D;
  Buffers B;
  sdd_params prm;
  cudaStream_t st;
  PhiloxKey key;
  float inv_tau_p, inv_tau_q;
  int steps_done;              // -1: no draft in progress; 0..T: denoising evaluations done this round
  uint64_t rounds, launches;
  std::vector<int> prompt_len, c_ub;
  int* mirror;                 // pinned mapped host memory [1 + 2 B + 1]
  int* mirror_dev;
  std::vector<cudaEvent_t> ev;
  int runahead;
  int lcap;                    // padded rows per sequence of the current round's drafter forwards
  size_t act_elems, xf_elems;  // capacity (elements) of the xn / att buffers (mlp: 4x) and of xf
  Net A;                       // autoregressive drafter of the speculative-decoding warm start (sdd_sps_attach)
  bool has_ar;
  void* ar_kv;                 // its KV cache [layer][batch][n_ctx][2][d] (layout as the target's)
  int* ar_eff;                 // [batch] effective length of its evaluation in flight
  bool sps_allowed;            // false once a round of another kind has run (the drafter's cache would have holes)
  int slot_prune;              // SDD_SLOT_PRUNE: 1 / 0 = the drafter's last block runs on the slot rows only / on all rows;
                               // unset (-1): on for forwards of 2048 rows or more (below that the forward is bound by
                               // launch latency and the extra gather launch costs what the smaller GEMMs save)
  bool cache_skip;             // SDD_CACHE_SKIP != 0 (default): skip drafter evaluations whose input did not change
  bool hilo;                   // SDD_HILO != 0 (default): hi/lo activation pairs in the target's MLP and LM head
  bool force_simt;             // SDD_GEMM=simt: run bf16 GEMMs on the CUDA-core kernel (cross-check)
  int bn_hint;                 // SDD_GEMM_BN: N tile of the tensor-core GEMM (0 = choose)
  bool head_stats;             // SDD_HEAD_STATS != 0 (default): soft-max statistics from the target LM head's epilogue
  bool use_graph;              // SDD_GRAPH != 0: sdd_step replays a captured graph per row-count bucket
  struct GraphEntry { cudaGraphExec_t exec; uint64_t launches; };
  std::map<std::tuple<int, void*, void*>, GraphEntry> graphs;
  std::vector<std::tuple<int, void*, void*>> prof_graphs;   // one-off graphs of the current timing pass
  // optional per-launch timing
  bool profiling;
  std::vector<cudaEvent_t> prof_ev;   // pairs (before, after)
  std::vector<int> prof_cat;
  size_t prof_used;
};

// RAII helper: brackets one launch with events when profiling is on
struct ProfScope {
  sdd_ctx* c;
  bool on;
  ProfScope(sdd_ctx* c_, int cat) : c(c_), on(false) {
    if (!c->profiling) return;
    if (c->prof_used + 2 > c->prof_ev.size()) {
      for (int i = 0; i < 2; ++i) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        c->prof_ev.push_back(e);
      }
    }
    record(c->prof_ev[c->prof_used]);
    c->prof_cat.push_back(cat);
    on = true;
  }
  ~ProfScope() {
    if (!on) return;
    record(c->prof_ev[c->prof_used + 1]);
    c->prof_used += 2;
  }
  // inside a stream capture a plain record only orders work; the external flag makes it a graph node that stamps
  // the event when the graph runs
  void record(cudaEvent_t e) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    cudaStreamIsCapturing(c->st, &cs);
    cudaEventRecordWithFlags(e, c->st, cs == cudaStreamCaptureStatusActive ? cudaEventRecordExternal : cudaEventRecordDefault);
  }
};

// ---- argument checks shared by workspace_bytes and create -------------------------------------
static int check_params(const sdd_model* target, const sdd_model* drafter, const sdd_params* p, Net* P, Net* Q) {
  if (p == nullptr) return SDD_E_ARG;
  SDD_TRY(parse_model(target, 1, P));
  SDD_TRY(parse_model(drafter, 0, Q));
  if (P->vocab != Q->vocab || P->dtype != Q->dtype) return SDD_E_SHAPE;
  if (p->gamma < 1 || p->gamma > 256 || p->T < 1 || p->T > 255 || p->batch < 1 || p->batch > 65535 || p->max_new < 1)
    return SDD_E_ARG;
  if (!(p->temp_p >= 0.f) || !(p->temp_q >= 0.f) || ((p->temp_p == 0.f) != (p->temp_q == 0.f))) return SDD_E_ARG;
  return SDD_OK;
}

static void fill_dims(const Net& P, const Net& Q, const sdd_params* p, int max_prompt, Dims* D) {
  D->batch = p->batch; D->gamma = p->gamma; D->T = p->T; D->max_new = p->max_new; D->V = P.vocab;
  D->tok_stride = P.n_ctx < Q.n_ctx ? P.n_ctx : Q.n_ctx;
  D->chunks = stats_chunks_for(P.vocab);
  D->chunks_cap = head_stats_chunks_max(P.vocab) > D->chunks ? head_stats_chunks_max(P.vocab) : D->chunks;
  int lmax = max_prompt + p->max_new + p->gamma;
  if (lmax > D->tok_stride) lmax = D->tok_stride;
  D->lcap_max = (int)align_up((size_t)lmax, ROW_TILE);
  D->rows_q = (long long)p->batch * D->lcap_max;
  const long long ver = (long long)p->batch * (p->gamma + 1), pre = (long long)p->batch * (max_prompt > 1 ? max_prompt - 1 : 0);
  D->rows_p = ver > pre ? ver : pre;
  D->max_prompt = max_prompt;
  D->esize = P.dtype == SDD_BF16 ? 2 : 4;
}

// ---- GEMM dispatch ----------------------------------------------------------------------------
// `a_elems` is the capacity of the A buffer in elements (the tensor map of an activation buffer covers all of it)
template <typename T>
static int gemm(sdd_ctx* c, int cat, const void* A, size_t a_elems, const void* W, const float* bias, long long M, int N,
                int K, int epi, void* out, int ldc, const QkvDst* qd = nullptr, const void* A_lo = nullptr,
                void* out_lo = nullptr, const int* skip = nullptr, const HeadStats* stats = nullptr, int* stats_chunks = nullptr) {
  if (stats_chunks != nullptr) *stats_chunks = 0;
  if (M <= 0) return SDD_OK;
  ProfScope prof(c, cat);
  c->launches++;
  if (std::is_same<T, __nv_bfloat16>::value && !c->force_simt) {
    SDD_CUDA(launch_gemm_tc((const __nv_bfloat16*)A, (long long)(a_elems / (size_t)K), (const __nv_bfloat16*)W, bias, (int)M,
                            N, K, epi, out, ldc, c->bn_hint, &c->B.rs->status, c->st, qd, (const __nv_bfloat16*)A_lo, out_lo, skip,
                            c->head_stats ? stats : nullptr, stats_chunks));
  } else {
    SDD_CUDA(launch_gemm_simt<T>((const T*)A, K, (const T*)W, bias, (int)M, N, K, epi, out, ldc, c->st, skip));
  }
  return SDD_OK;
}

// the tensor-core path (tcgen05 GEMMs with the fused QKV epilogue + tensor-core attention) needs bf16 and d_head 64
template <typename T>
static bool use_tc(const sdd_ctx* c, const Net& N) {
  return std::is_same<T, __nv_bfloat16>::value && !c->force_simt && N.d_head == 64;
}

#define SDD_LAUNCH(c, cat, expr) \
  do {                           \
    ProfScope prof__((c), (cat)); \
    (c)->launches++;             \
    SDD_CUDA(expr);              \
  } while (0)

// one transformer block on `rows` rows; attention is issued by the caller-supplied functor
// slot_rows > 0 (drafter): after the last block's attention only the slot rows go on (gathered by `gather` into the
// head of the dead qkv buffer and into h_s), because nothing else reaches the LM head
template <typename T, typename QkvFn, typename AttnFn, typename GatherFn>
static int run_blocks(sdd_ctx* c, const Net& N, long long rows, int gcat, bool hilo_mlp, const int* skip, QkvFn qkv_dst,
                      AttnFn attn, long long slot_rows, GatherFn gather, bool first_ln_done = false) {
  const Buffers& B = c->B;
  const int d = N.d;
  for (int l = 0; l < N.n_layer; ++l) {
    const Layer& L = N.layers[l];
    const bool pruned = slot_rows > 0 && l == N.n_layer - 1;
    // first_ln_done: the embedding kernel has already written the first block's LayerNorm to xn
    if (!(l == 0 && first_ln_done))
      SDD_LAUNCH(c, CAT_LAYERNORM, launch_layernorm<T>(B.h, L.ln1_g, L.ln1_b, (T*)B.xn, rows, d, c->st, nullptr, skip));
    QkvDst qd = {};
    const bool fused = qkv_dst(l, &qd);
    SDD_TRY(gemm<T>(c, gcat, B.xn, c->act_elems, L.w_qkv, L.b_qkv, rows, 3 * d, d, fused ? EPI_QKV : EPI_STORE, B.qkv,
                    3 * d, fused ? &qd : nullptr, nullptr, nullptr, skip));
    SDD_TRY(attn(l));
    if (pruned) {
      SDD_TRY(gather());
      SDD_TRY(gemm<T>(c, gcat, B.qkv, 3 * c->act_elems, L.w_o, L.b_o, slot_rows, d, d, EPI_RESIDUAL, B.h_s, d, nullptr, nullptr,
                      nullptr, skip));
      SDD_LAUNCH(c, CAT_LAYERNORM, launch_layernorm<T>(B.h_s, L.ln2_g, L.ln2_b, (T*)B.xn, slot_rows, d, c->st, nullptr, skip));
      SDD_TRY(gemm<T>(c, gcat, B.xn, c->act_elems, L.w_fc1, L.b_fc1, slot_rows, 4 * d, d, EPI_GELU, B.mlp, 4 * d, nullptr,
                      nullptr, nullptr, skip));
      SDD_TRY(gemm<T>(c, gcat, B.mlp, 4 * c->act_elems, L.w_fc2, L.b_fc2, slot_rows, d, 4 * d, EPI_RESIDUAL, B.h_s, d, nullptr,
                      nullptr, nullptr, skip));
      break;
    }
    SDD_TRY(gemm<T>(c, gcat, B.att, c->act_elems, L.w_o, L.b_o, rows, d, d, EPI_RESIDUAL, B.h, d, nullptr, nullptr, nullptr, skip));
    // hilo_mlp: the MLP's two products take their activations as hi/lo bf16 pairs (see sdd_gemm_tc.cu)
    T* xn_lo = hilo_mlp ? (T*)B.xn_lo : nullptr;
    void* mlp_lo = hilo_mlp ? B.mlp_lo : nullptr;
    SDD_LAUNCH(c, CAT_LAYERNORM, launch_layernorm<T>(B.h, L.ln2_g, L.ln2_b, (T*)B.xn, rows, d, c->st, xn_lo, skip));
    SDD_TRY(gemm<T>(c, gcat, B.xn, c->act_elems, L.w_fc1, L.b_fc1, rows, 4 * d, d, EPI_GELU, B.mlp, 4 * d, nullptr, xn_lo,
                    mlp_lo, skip));
    SDD_TRY(gemm<T>(c, gcat, B.mlp, 4 * c->act_elems, L.w_fc2, L.b_fc2, rows, d, 4 * d, EPI_RESIDUAL, B.h, d, nullptr, mlp_lo, nullptr,
                    skip));
  }
  return SDD_OK;
}

// one drafter evaluation M_q([x_{0:i}] ∘ [slots]) -> step_logits[B, gamma, V]
template <typename T>
static int forward_drafter(sdd_ctx* c) {
  const Net& Q = c->Q;
  const Buffers& B = c->B;
  const Dims& D = c->D;
  const int lcap = c->lcap;
  const long long rows = (long long)D.batch * lcap;
  // every kernel of the evaluation returns at once when the previous step revealed nothing (RoundState.skip_forward)
  const int* skip = &B.rs->skip_forward;
  const long long slot_rows = (long long)D.batch * D.gamma;
  const bool prune = c->slot_prune == 1 || (c->slot_prune < 0 && rows >= 2048);
  SDD_LAUNCH(c, CAT_GLUE, launch_embed_drafter<T>((const T*)Q.wte, (const T*)Q.wpe, B.tokens, D.tok_stride, B.ctx_len, B.slot_ids,
                                        D.batch, D.gamma, lcap, Q.d, B.h, c->st, skip, Q.layers[0].ln1_g, Q.layers[0].ln1_b,
                                        (T*)B.xn, Q.vocab, &B.rs->status));
  const bool tc = use_tc<T>(c, Q);
  SDD_TRY((run_blocks<T>(c, Q, rows, CAT_GEMM_Q, false, skip,
    [&](int, QkvDst* qd) -> bool {
      if (!tc) return false;
      qd->k_dst = nullptr; qd->vt_dst = (__nv_bfloat16*)B.vt; qd->ctx_len = B.ctx_len; qd->rows_per_seq = lcap;
      qd->mode = 0; qd->d = Q.d; qd->k_seq_rows = 0; qd->vt_ld = D.lcap_max;
      return true;
    },
    [&](int) -> int {
      if (tc) {
        const __nv_bfloat16* qkv = (const __nv_bfloat16*)B.qkv;
        SDD_LAUNCH(c, CAT_ATTN_Q, launch_attn_tc(qkv, (long long)(c->act_elems / Q.d), 3 * Q.d, 0, qkv,
                                                 (long long)(c->act_elems / Q.d), 3 * Q.d, Q.d, lcap,
                                                 (const __nv_bfloat16*)B.vt, D.lcap_max, (__nv_bfloat16*)B.att, Q.d, B.ctx_len,
                                                 D.batch, Q.n_head, Q.d, D.gamma, 0, lcap, &B.rs->status, c->st, skip));
      } else {
        SDD_LAUNCH(c, CAT_ATTN_Q, launch_attn_bidir<T>((const T*)B.qkv, (T*)B.att, B.ctx_len, D.batch, D.gamma, lcap, Q.n_head,
                                                       Q.d_head, c->st, skip));
      }
      return SDD_OK;
    },
    prune ? slot_rows : 0,
    [&]() -> int {
      SDD_LAUNCH(c, CAT_GLUE, launch_gather_slots<T>((const T*)B.att, B.h, B.ctx_len, D.batch, D.gamma, lcap, Q.d, (T*)B.qkv,
                                                     B.h_s, c->st, skip));
      return SDD_OK;
    },
    true)));
  if (prune)
    SDD_LAUNCH(c, CAT_LAYERNORM, launch_layernorm<T>(B.h_s, Q.lnf_g, Q.lnf_b, (T*)B.xf, slot_rows, Q.d, c->st, nullptr, skip));
  else
    SDD_LAUNCH(c, CAT_LAYERNORM, launch_layernorm_slots<T>(B.h, Q.lnf_g, Q.lnf_b, (T*)B.xf, B.ctx_len, D.batch, D.gamma, lcap, Q.d,
                                                           c->st, skip));
  SDD_TRY(gemm<T>(c, CAT_HEAD_Q, B.xf, c->xf_elems, Q.wte, nullptr, (long long)D.batch * D.gamma, D.V, Q.d, EPI_STORE_F32, B.step_logits, D.V,
                  nullptr, nullptr, nullptr, skip));
  return SDD_OK;
}

// Causal forward of network N over rows_per_seq new tokens per sequence against its KV cache `kv`; `len` holds the
// per-sequence length that fixes the rows' positions (see TargetMode); the caller has written the embeddings to B.h.
template <typename T>
static int forward_causal(sdd_ctx* c, const Net& N, void* kv, const int* len, int mode, int rows_per_seq, bool lm_head,
                          float* logits_out, bool hilo, int gcat, int hcat, int acat, const HeadStats* stats = nullptr,
                          int* stats_chunks = nullptr) {
  const Buffers& B = c->B;
  const Dims& D = c->D;
  const long long rows = (long long)D.batch * rows_per_seq;
  const size_t layer_elems = (size_t)D.batch * N.n_ctx * 2 * N.d;
  const bool tc = use_tc<T>(c, N);
  hilo = hilo && tc;
  // tensor-core path: per layer the cache is K [B][n_ctx][d] followed by V^T [B][d][n_ctx];
  // CUDA-core path: [B][n_ctx][K|V][d]
  SDD_TRY((run_blocks<T>(c, N, rows, gcat, hilo, nullptr,
    [&](int l, QkvDst* qd) -> bool {
      if (!tc) return false;
      __nv_bfloat16* kc = (__nv_bfloat16*)kv + (size_t)l * layer_elems;
      qd->k_dst = kc; qd->vt_dst = kc + layer_elems / 2; qd->ctx_len = len; qd->rows_per_seq = rows_per_seq;
      qd->mode = mode == TARGET_VERIFY ? 1 : 2; qd->d = N.d; qd->k_seq_rows = N.n_ctx; qd->vt_ld = N.n_ctx;
      return true;
    },
    [&](int l) -> int {
      T* cache = (T*)kv + (size_t)l * layer_elems;
      if (tc) {
        const __nv_bfloat16* kc = (const __nv_bfloat16*)cache;
        SDD_LAUNCH(c, acat, launch_attn_tc((const __nv_bfloat16*)B.qkv, (long long)(c->act_elems / N.d), 3 * N.d, 0, kc,
                                           (long long)D.batch * N.n_ctx, N.d, 0, N.n_ctx, kc + layer_elems / 2, N.n_ctx,
                                           (__nv_bfloat16*)B.att, N.d, len, D.batch, N.n_head, N.d, D.gamma,
                                           mode == TARGET_VERIFY ? 1 : 2, rows_per_seq, &B.rs->status, c->st));
      } else {
        SDD_LAUNCH(c, CAT_GLUE, launch_kv_append<T>((const T*)B.qkv, cache, len, D.batch, rows_per_seq, mode, N.n_ctx, N.d,
                                                    c->st));
        SDD_LAUNCH(c, acat, launch_attn_cached<T>((const T*)B.qkv, cache, (T*)B.att, len, D.batch, rows_per_seq, mode,
                                                  N.n_ctx, N.n_head, N.d_head, c->st));
      }
      return SDD_OK;
    },
    0, []() -> int { return SDD_OK; })));
  if (lm_head) {
    T* xf_lo = hilo ? (T*)B.xf_lo : nullptr;
    SDD_LAUNCH(c, CAT_LAYERNORM, launch_layernorm<T>(B.h, N.lnf_g, N.lnf_b, (T*)B.xf, rows, N.d, c->st, xf_lo));
    SDD_TRY(gemm<T>(c, hcat, B.xf, c->xf_elems, N.wte, nullptr, rows, D.V, N.d, EPI_STORE_F32, logits_out, D.V, nullptr,
                    xf_lo, nullptr, nullptr, stats, stats_chunks));
  }
  return SDD_OK;
}

// target forward over rows_per_seq new tokens per sequence against the KV cache
template <typename T>
static int forward_target(sdd_ctx* c, int mode, int rows_per_seq, bool lm_head, const HeadStats* stats = nullptr,
                          int* stats_chunks = nullptr) {
  const Net& P = c->P;
  const Buffers& B = c->B;
  const Dims& D = c->D;
  if (rows_per_seq <= 0) return SDD_OK;
  // a verification forward carries the round's own draft length (gamma + 1 rows); slot_ids is [batch][that length]
  const int slot_stride = mode == TARGET_VERIFY ? rows_per_seq - 1 : D.gamma;
  SDD_LAUNCH(c, CAT_GLUE, launch_embed_target<T>((const T*)P.wte, (const T*)P.wpe, B.tokens, D.tok_stride, B.ctx_len, B.slot_ids,
                                       D.batch, slot_stride, rows_per_seq, mode, P.d, B.h, c->st, P.vocab, &B.rs->status));
  return forward_causal<T>(c, P, B.kv, B.ctx_len, mode, rows_per_seq, lm_head, B.logits_p, c->hilo, CAT_GEMM_P, CAT_HEAD_P,
                           CAT_ATTN_P, stats, stats_chunks);
}

// One evaluation of the autoregressive drafter of a speculative-decoding round, producing the logits of slot j
// (Section "Preliminaries and Settings", paragraph "Speculative decoding": gamma sequential evaluations of M_q).
// Evaluation 0 feeds positions c-2 and c-1: after a round that accepted every draft the drafter has never seen the
// last draft token, and recomputing position c-2 otherwise reproduces what the cache already holds.  Evaluation
// j > 0 feeds draft j-1 at position c+j-1.  The logits go to the head of the logits_p buffer, which is free until
// the verification forward.
template <typename T>
static int forward_ar_drafter(sdd_ctx* c, int gamma, int j) {
  const Net& A = c->A;
  const Buffers& B = c->B;
  const Dims& D = c->D;
  const int rows = j == 0 ? 2 : 1, off = j == 0 ? -1 : j;
  SDD_LAUNCH(c, CAT_GLUE, launch_embed_ar<T>((const T*)A.wte, (const T*)A.wpe, B.tokens, D.tok_stride, B.ctx_len, B.slot_ids,
                                             D.batch, gamma, rows, off, A.d, B.h, c->ar_eff, c->st, A.vocab, &B.rs->status));
  SDD_TRY(forward_causal<T>(c, A, c->ar_kv, c->ar_eff, TARGET_VERIFY, rows, true, B.logits_p, false, CAT_GEMM_Q, CAT_HEAD_Q,
                            CAT_ATTN_Q));
  SDD_LAUNCH(c, CAT_SAMPLE, launch_ar_sample(B.logits_p, rows, B.slot_ids, B.q_logits, B.logq, B.lse_q, B.reveal_step, D.batch,
                                             gamma, j, D.V, c->inv_tau_q, c->key, B.rs, c->st));
  return SDD_OK;
}

// refresh the host's upper bound of every context length from the pinned mirror and pick the
// padded row count of this round's drafter forwards
static void choose_lcap(sdd_ctx* c) {
  const int Bn = c->D.batch;
  // the commit kernel writes head stamp, body, tail stamp; a reader therefore takes the tail first and the head
  // last: equal stamps then bracket a body that no writer touched in between
  volatile int* m = c->mirror;
  const int s1 = m[1 + 2 * Bn];
  std::atomic_thread_fence(std::memory_order_acquire);
  std::vector<int> seen(Bn);
  for (int b = 0; b < Bn; ++b) seen[b] = m[1 + b];
  std::atomic_thread_fence(std::memory_order_acquire);
  const int s0 = m[0];
  const int per_round = c->D.gamma + 1;
  if (s0 == s1 && s1 > 0 && (uint64_t)s1 <= c->rounds) {
    const long long behind = (long long)c->rounds - s1;
    for (int b = 0; b < Bn; ++b) {
      long long ub = seen[b] + behind * per_round;
      if (ub < c->c_ub[b]) c->c_ub[b] = (int)ub;
    }
  }
  int cmax = 1;
  for (int b = 0; b < Bn; ++b) {
    const int cap = c->prompt_len[b] + c->D.max_new;
    if (c->c_ub[b] > cap) c->c_ub[b] = cap;
    if (c->c_ub[b] > cmax) cmax = c->c_ub[b];
  }
  int lcap = (int)align_up((size_t)(cmax + c->D.gamma), ROW_TILE);
  if (lcap > c->D.lcap_max) lcap = c->D.lcap_max;
  c->lcap = lcap;
}

template <typename T>
static int draft_step_t(sdd_ctx* c) {
  const Buffers& B = c->B;
  const Dims& D = c->D;
  const int k = D.T - c->steps_done;
  SDD_TRY(forward_drafter<T>(c));
  SDD_LAUNCH(c, CAT_SAMPLE, launch_unmask_sample(B.step_logits, B.slot_ids, B.q_logits, B.logq, B.lse_q, B.reveal_step, D.batch,
                                     D.gamma, D.V, k, c->inv_tau_q, c->key, B.rs, c->cache_skip ? 1 : 0, c->st));
  c->steps_done++;
  return SDD_OK;
}

template <typename T>
static int verify_accept_t(sdd_ctx* c, int gamma, int32_t* out_ids, int32_t* n_out) {
  // gamma = the round's draft length; gamma = 0 is plain autoregressive decoding of the target: one token is fed,
  // nothing is tested, and the extra token is the draw from p (Algorithm 1 with an empty draft)
  const Buffers& B = c->B;
  const Dims& D = c->D;
  // the rows' soft-max statistics come out of the LM head's epilogue where that runs on a persistent tensor-core
  // kernel (chunks > 0); otherwise a pass over the logits produces them
  const HeadStats hs = {c->inv_tau_p, B.partial_p, D.chunks_cap};
  int chunks = 0;
  SDD_TRY(forward_target<T>(c, TARGET_VERIFY, gamma + 1, true, &hs, &chunks));
  if (chunks == 0) {
    SDD_LAUNCH(c, CAT_STATS, launch_row_stats(B.logits_p, (long long)D.batch * (gamma + 1), nullptr, 0, D.V, c->inv_tau_p, 0.f,
                                   B.partial_p, c->st));
    chunks = D.chunks;
  }
  SDD_LAUNCH(c, CAT_ACCEPT, launch_accept(B.logits_p, B.q_logits, B.slot_ids, B.logq, B.lse_q, B.partial_p, chunks, nullptr, 0, D.batch, gamma, D.V,
                              c->inv_tau_p, c->inv_tau_p == 0.f ? 0.f : 1.f, c->key, 0u, B.rs, B.accept_prob, B.n_accept,
                              B.extra_token, nullptr, c->st));
  SDD_LAUNCH(c, CAT_COMMIT, launch_commit(B.tokens, D.tok_stride, B.ctx_len, B.n_emitted, B.slot_ids, B.n_accept, B.extra_token,
                              D.batch, gamma, D.max_new, B.rs, out_ids, n_out, c->mirror_dev, c->st));
  return SDD_OK;
}

// =================================================================================================
extern "C" {

int32_t sdd_workspace_bytes(const sdd_model* target, const sdd_model* drafter, const sdd_params* params,
                            uint64_t* out_bytes) {
  if (out_bytes == nullptr) return SDD_E_ARG;
  Net P, Q;
  SDD_TRY(check_params(target, drafter, params, &P, &Q));
  // without the prompt lengths the drafter may have to cover its whole position table
  Dims D;
  const int tok_stride = P.n_ctx < Q.n_ctx ? P.n_ctx : Q.n_ctx;
  fill_dims(P, Q, params, tok_stride, &D);
  *out_bytes = carve(D, P, Q, nullptr, nullptr);
  return SDD_OK;
}

static int load_prompts(sdd_ctx* c, const int32_t* prompt_ids, int32_t prompt_stride, const int32_t* prompt_len, int max_prompt);
static int prefill_ar_drafter(sdd_ctx* c);

int32_t sdd_create(const sdd_model* target, const sdd_model* drafter, const sdd_params* params,
                   const int32_t* prompt_ids, int32_t prompt_stride, const int32_t* prompt_len, void* workspace,
                   uint64_t workspace_bytes, sdd_ctx** out) {
  if (out == nullptr || prompt_ids == nullptr || prompt_len == nullptr || workspace == nullptr) return SDD_E_ARG;
  *out = nullptr;
  sdd_ctx* c = new (std::nothrow) sdd_ctx();
  if (c == nullptr) return SDD_E_ARG;
  struct Guard { sdd_ctx* c; ~Guard() { if (c) sdd_destroy(c); } } guard{c};
  c->mirror = nullptr;
  int s = check_params(target, drafter, params, &c->P, &c->Q);
  if (s != SDD_OK) return s;
  int max_prompt = 0;
  for (int b = 0; b < params->batch; ++b) {
    if (prompt_len[b] < 1 || prompt_len[b] > prompt_stride) return SDD_E_ARG;
    if (prompt_len[b] > max_prompt) max_prompt = prompt_len[b];
  }
  const int tok_stride = c->P.n_ctx < c->Q.n_ctx ? c->P.n_ctx : c->Q.n_ctx;
  if ((long long)max_prompt + params->max_new + params->gamma > tok_stride) return SDD_E_CTX_FULL;
  // the layout is the one sdd_workspace_bytes reports (prompt-independent), so its size check is exact
  fill_dims(c->P, c->Q, params, tok_stride, &c->D);
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SDD_E_WORKSPACE;
  if (carve(c->D, c->P, c->Q, nullptr, nullptr) > workspace_bytes) return SDD_E_WORKSPACE;
  carve(c->D, c->P, c->Q, (uint8_t*)workspace, &c->B);
  c->prm = *params;
  c->st = (cudaStream_t)params->stream;
  c->key = make_key(params->seed);
  c->inv_tau_p = params->temp_p > 0.f ? 1.f / params->temp_p : 0.f;
  c->inv_tau_q = params->temp_q > 0.f ? 1.f / params->temp_q : 0.f;
  c->steps_done = -1;
  c->rounds = 0;
  c->launches = 0;
  c->has_ar = false;
  c->ar_kv = nullptr;
  c->ar_eff = nullptr;
  c->sps_allowed = true;
  c->profiling = false;
  c->prof_used = 0;
  {
    const size_t rq = (size_t)c->D.rows_q, rp = (size_t)c->D.rows_p;
    const size_t a = rq * c->Q.d, b = rp * c->P.d;
    c->act_elems = a > b ? a : b;
    c->xf_elems = (size_t)params->batch * (params->gamma + 1) * (c->Q.d > c->P.d ? c->Q.d : c->P.d);
    const char* g = getenv("SDD_GEMM");
    c->force_simt = g != nullptr && strcmp(g, "simt") == 0;
    const char* cs = getenv("SDD_CACHE_SKIP");
    c->cache_skip = cs == nullptr || atoi(cs) != 0;
    const char* sp = getenv("SDD_SLOT_PRUNE");
    c->slot_prune = sp == nullptr ? -1 : (atoi(sp) != 0 ? 1 : 0);
    const char* hl = getenv("SDD_HILO");
    c->hilo = hl == nullptr || atoi(hl) != 0;
    const char* bn = getenv("SDD_GEMM_BN");
    c->bn_hint = bn ? atoi(bn) : 0;
    const char* hs = getenv("SDD_HEAD_STATS");
    c->head_stats = hs == nullptr || atoi(hs) != 0;
    const char* gr = getenv("SDD_GRAPH");
    // the legacy default stream cannot be captured: rounds are then enqueued kernel by kernel
    c->use_graph = (gr == nullptr || atoi(gr) != 0) && c->st != nullptr && c->st != cudaStreamLegacy;
  }
  c->prompt_len.assign(prompt_len, prompt_len + params->batch);
  c->c_ub = c->prompt_len;
  const char* ra = getenv("SDD_RUNAHEAD");
  c->runahead = ra ? atoi(ra) : 2;
  if (c->runahead < 1) c->runahead = 1;
  if (c->runahead > 8) c->runahead = 8;
  c->ev.resize(c->runahead + 1);
  for (auto& e : c->ev) e = nullptr;
  for (auto& e : c->ev) SDD_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  const size_t mirror_ints = 2 + 2 * (size_t)params->batch;
  SDD_CUDA(cudaHostAlloc((void**)&c->mirror, mirror_ints * sizeof(int), cudaHostAllocMapped));
  memset(c->mirror, 0, mirror_ints * sizeof(int));
  SDD_CUDA(cudaHostGetDevicePointer((void**)&c->mirror_dev, c->mirror, 0));

  if (c->P.dtype == SDD_BF16) {   // before anything can be captured into a graph
    SDD_CUDA(tc_prepare_gemm());
    SDD_CUDA(tc_prepare_attn());
  }
  // the tensor-core attention multiplies masked probabilities (exact zeros) with whatever the V^T cache holds
  // past the valid positions, so that memory must be finite
  SDD_CUDA(cudaMemsetAsync(c->B.kv, 0, (size_t)c->P.n_layer * params->batch * c->P.n_ctx * 2 * c->P.d * c->D.esize, c->st));
  s = load_prompts(c, prompt_ids, prompt_stride, prompt_len, max_prompt);
  if (s != SDD_OK) return s;
  guard.c = nullptr;
  *out = c;
  return SDD_OK;
}

// start of a generation: zero the small state and the activations (padding rows must stay finite), load the prompts,
// prefill the target's KV cache with x_{0:c-2}
static int load_prompts(sdd_ctx* c, const int32_t* prompt_ids, int32_t prompt_stride, const int32_t* prompt_len, int max_prompt) {
  const Buffers& B = c->B;
  const int batch = c->D.batch;
  const size_t state_bytes = (size_t)((uint8_t*)B.step_logits - (uint8_t*)B.rs);
  SDD_CUDA(cudaMemsetAsync(B.rs, 0, state_bytes, c->st));
  const size_t act_bytes = (size_t)((uint8_t*)B.kv - (uint8_t*)B.h);
  SDD_CUDA(cudaMemsetAsync(B.h, 0, act_bytes, c->st));
  SDD_CUDA(cudaMemcpy2DAsync(B.tokens, (size_t)c->D.tok_stride * 4, prompt_ids, (size_t)prompt_stride * 4,
                             (size_t)max_prompt * 4, batch, cudaMemcpyDeviceToDevice, c->st));
  SDD_CUDA(cudaMemcpyAsync(B.ctx_len, prompt_len, (size_t)batch * 4, cudaMemcpyHostToDevice, c->st));
  c->D.max_prompt = max_prompt;
  int s;
  if (c->P.dtype == SDD_BF16) s = forward_target<__nv_bfloat16>(c, TARGET_PREFILL, max_prompt - 1, false);
  else s = forward_target<float>(c, TARGET_PREFILL, max_prompt - 1, false);
  if (s != SDD_OK) return s;
  // prompt_len is host memory owned by the caller: make sure the copy above has consumed it
  SDD_CUDA(cudaStreamSynchronize(c->st));
  return SDD_OK;
}

// A new generation in the same context: same models, parameters, workspace and captured graphs; new prompts.
int32_t sdd_reset(sdd_ctx* c, const int32_t* prompt_ids, int32_t prompt_stride, const int32_t* prompt_len) {
  if (c == nullptr || prompt_ids == nullptr || prompt_len == nullptr) return SDD_E_ARG;
  if (c->steps_done != -1) return SDD_E_STATE;
  const int batch = c->D.batch;
  int max_prompt = 0;
  for (int b = 0; b < batch; ++b) {
    if (prompt_len[b] < 1 || prompt_len[b] > prompt_stride) return SDD_E_ARG;
    if (c->has_ar && prompt_len[b] < 2) return SDD_E_ARG;
    if (prompt_len[b] > max_prompt) max_prompt = prompt_len[b];
  }
  if ((long long)max_prompt + c->D.max_new + c->D.gamma > c->D.tok_stride) return SDD_E_CTX_FULL;
  if (c->has_ar && (long long)max_prompt + c->D.max_new + c->D.gamma > c->A.n_ctx) return SDD_E_CTX_FULL;
  // everything enqueued for the old generation has to be over before the host-side round bookkeeping restarts
  SDD_CUDA(cudaStreamSynchronize(c->st));
  c->rounds = 0;
  c->steps_done = -1;
  c->sps_allowed = true;
  c->prompt_len.assign(prompt_len, prompt_len + batch);
  c->c_ub = c->prompt_len;
  memset(c->mirror, 0, (2 + 2 * (size_t)batch) * sizeof(int));
  SDD_TRY(load_prompts(c, prompt_ids, prompt_stride, prompt_len, max_prompt));
  if (c->has_ar) SDD_TRY(prefill_ar_drafter(c));
  return SDD_OK;
}

// ---- round pieces: host bookkeeping outside, stream work inside (the latter can be captured in a graph) ----
static int round_prologue(sdd_ctx* c) {
  // bound the host's run-ahead so that the length mirror stays fresh
  if (c->rounds >= (uint64_t)c->runahead)
    SDD_CUDA(cudaEventSynchronize(c->ev[(c->rounds - c->runahead) % c->ev.size()]));
  choose_lcap(c);
  return SDD_OK;
}
static int enqueue_draft_begin(sdd_ctx* c) {
  // per-launch timing: a few empty event pairs per round measure what a pair costs by itself (subtracted later)
  for (int i = 0; i < 4 && c->profiling; ++i) { ProfScope calib(c, CAT_COUNT); }
  SDD_LAUNCH(c, CAT_GLUE, launch_reset_slots(c->B.slot_ids, c->B.reveal_step, c->D.batch * c->D.gamma, c->D.V, c->B.rs, c->st));
  c->steps_done = 0;
  return SDD_OK;
}
static int enqueue_draft_step(sdd_ctx* c) {
  return c->P.dtype == SDD_BF16 ? draft_step_t<__nv_bfloat16>(c) : draft_step_t<float>(c);
}
static int enqueue_verify_accept(sdd_ctx* c, int gamma, int32_t* out_ids, int32_t* n_out) {
  return c->P.dtype == SDD_BF16 ? verify_accept_t<__nv_bfloat16>(c, gamma, out_ids, n_out)
                                : verify_accept_t<float>(c, gamma, out_ids, n_out);
}
static int round_epilogue(sdd_ctx* c, int max_emitted) {
  SDD_CUDA(cudaEventRecord(c->ev[c->rounds % c->ev.size()], c->st));
  c->rounds++;
  c->steps_done = -1;
  for (auto& ub : c->c_ub) ub += max_emitted;
  return SDD_OK;
}

int32_t sdd_draft_begin(sdd_ctx* c) {
  if (c == nullptr) return SDD_E_ARG;
  c->sps_allowed = false;
  SDD_TRY(round_prologue(c));
  return enqueue_draft_begin(c);
}

int32_t sdd_draft_step(sdd_ctx* c) {
  if (c == nullptr) return SDD_E_ARG;
  if (c->steps_done < 0 || c->steps_done >= c->D.T) return SDD_E_STATE;
  return enqueue_draft_step(c);
}

int32_t sdd_draft(sdd_ctx* c) {
  SDD_TRY(sdd_draft_begin(c));
  for (int i = 0; i < c->D.T; ++i) SDD_TRY(sdd_draft_step(c));
  return SDD_OK;
}

int32_t sdd_verify_accept(sdd_ctx* c, int32_t* out_ids, int32_t* n_out) {
  if (c == nullptr) return SDD_E_ARG;
  if (c->steps_done != c->D.T) return SDD_E_STATE;
  SDD_TRY(enqueue_verify_accept(c, c->D.gamma, out_ids, n_out));
  return round_epilogue(c, c->D.gamma + 1);
}

// One whole round.  Every launch parameter of a round is fixed for a given padded row count (all lengths,
// the round index and the RNG state live on the device), so the round is captured once per row-count bucket
// and replayed as a CUDA graph; SDD_GRAPH=0 (or per-launch timing) enqueues the kernels one by one instead.
int32_t sdd_step(sdd_ctx* c, int32_t* out_ids, int32_t* n_out) {
  if (c == nullptr) return SDD_E_ARG;
  if (c->steps_done != -1) return SDD_E_STATE;
  c->sps_allowed = false;
  if (!c->use_graph) {
    SDD_TRY(sdd_draft(c));
    return sdd_verify_accept(c, out_ids, n_out);
  }
  SDD_TRY(round_prologue(c));
  // per-launch timing: the event pairs are captured into a one-off graph, so the stamps are taken on the device
  // timeline without host launch gaps in between
  const auto key = std::make_tuple(c->profiling ? -c->lcap - (int)c->prof_graphs.size() - 1 : c->lcap, (void*)out_ids,
                                   (void*)n_out);
  auto it = c->graphs.find(key);
  if (it == c->graphs.end()) {
    const uint64_t l0 = c->launches;
    SDD_CUDA(cudaStreamBeginCapture(c->st, cudaStreamCaptureModeThreadLocal));
    int s = enqueue_draft_begin(c);
    for (int i = 0; i < c->D.T && s == SDD_OK; ++i) s = enqueue_draft_step(c);
    if (s == SDD_OK) s = enqueue_verify_accept(c, c->D.gamma, out_ids, n_out);
    cudaGraph_t g = nullptr;
    cudaError_t e = cudaStreamEndCapture(c->st, &g);
    c->steps_done = -1;
    if (s != SDD_OK) { if (g) cudaGraphDestroy(g); return s; }
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamEndCapture");
    sdd_ctx::GraphEntry ge;
    ge.exec = nullptr;
    ge.launches = c->launches - l0;
    c->launches = l0;
    e = cudaGraphInstantiate(&ge.exec, g, 0);
    cudaGraphDestroy(g);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGraphInstantiate");
    it = c->graphs.emplace(key, ge).first;
    if (c->profiling) c->prof_graphs.push_back(key);
  }
  SDD_CUDA(cudaGraphLaunch(it->second.exec, c->st));
  c->launches += it->second.launches;
  return round_epilogue(c, c->D.gamma + 1);
}

// Plain autoregressive decoding of the target (the baseline of Table 1): a round with an empty draft.
int32_t sdd_ar_step(sdd_ctx* c, int32_t* out_ids, int32_t* n_out) {
  if (c == nullptr) return SDD_E_ARG;
  if (c->steps_done != -1) return SDD_E_STATE;
  c->sps_allowed = false;
  if (c->rounds >= (uint64_t)c->runahead)
    SDD_CUDA(cudaEventSynchronize(c->ev[(c->rounds - c->runahead) % c->ev.size()]));
  if (!c->use_graph || c->profiling) {
    SDD_TRY(enqueue_verify_accept(c, 0, out_ids, n_out));
    return round_epilogue(c, 1);
  }
  const auto key = std::make_tuple(0, (void*)out_ids, (void*)n_out);   // row count 0 never names a SpecDiff round
  auto it = c->graphs.find(key);
  if (it == c->graphs.end()) {
    const uint64_t l0 = c->launches;
    SDD_CUDA(cudaStreamBeginCapture(c->st, cudaStreamCaptureModeThreadLocal));
    const int s = enqueue_verify_accept(c, 0, out_ids, n_out);
    cudaGraph_t g = nullptr;
    cudaError_t e = cudaStreamEndCapture(c->st, &g);
    if (s != SDD_OK) { if (g) cudaGraphDestroy(g); return s; }
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamEndCapture");
    sdd_ctx::GraphEntry ge;
    ge.exec = nullptr;
    ge.launches = c->launches - l0;
    c->launches = l0;
    e = cudaGraphInstantiate(&ge.exec, g, 0);
    cudaGraphDestroy(g);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGraphInstantiate");
    it = c->graphs.emplace(key, ge).first;
  }
  SDD_CUDA(cudaGraphLaunch(it->second.exec, c->st));
  c->launches += it->second.launches;
  return round_epilogue(c, 1);
}

// ---- speculative-decoding warm start (Section "Sequence initialization") -------------------------
static size_t ar_workspace(const Net& A, int batch, size_t esize) {
  return align_up((size_t)A.n_layer * batch * A.n_ctx * 2 * A.d * esize, 256) + align_up((size_t)batch * 4, 256);
}

int32_t sdd_sps_workspace_bytes(const sdd_model* ar_drafter, const sdd_params* params, uint64_t* out_bytes) {
  if (out_bytes == nullptr || params == nullptr || params->batch < 1) return SDD_E_ARG;
  Net A;
  SDD_TRY(parse_model(ar_drafter, 1, &A));
  *out_bytes = ar_workspace(A, params->batch, A.dtype == SDD_BF16 ? 2 : 4);
  return SDD_OK;
}

int32_t sdd_sps_attach(sdd_ctx* c, const sdd_model* ar_drafter, void* workspace, uint64_t workspace_bytes) {
  if (c == nullptr || workspace == nullptr) return SDD_E_ARG;
  if (c->rounds != 0 || c->steps_done != -1 || c->has_ar) return SDD_E_STATE;
  Net A;
  SDD_TRY(parse_model(ar_drafter, 1, &A));
  // the drafter shares the activation buffers, which are sized for the target's verification rows
  if (A.vocab != c->P.vocab || A.dtype != c->P.dtype || A.d > c->P.d) return SDD_E_SHAPE;
  for (int p : c->prompt_len)
    if (p < 2) return SDD_E_ARG;                       // its first evaluation feeds positions c-2 and c-1
  if ((long long)c->D.max_prompt + c->D.max_new + c->D.gamma > A.n_ctx) return SDD_E_CTX_FULL;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || ar_workspace(A, c->D.batch, c->D.esize) > workspace_bytes)
    return SDD_E_WORKSPACE;
  c->A = A;
  const size_t kv_bytes = (size_t)A.n_layer * c->D.batch * A.n_ctx * 2 * A.d * c->D.esize;
  c->ar_kv = workspace;
  c->ar_eff = (int*)((uint8_t*)workspace + align_up(kv_bytes, 256));
  SDD_CUDA(cudaMemsetAsync(workspace, 0, ar_workspace(A, c->D.batch, c->D.esize), c->st));   // V^T past the valid positions must be finite
  int s = prefill_ar_drafter(c);
  if (s != SDD_OK) { c->ar_kv = nullptr; return s; }
  c->has_ar = true;
  return SDD_OK;
}

// prefill of the autoregressive drafter's cache with x_{0:c-2}, as for the target
static int prefill_ar_drafter(sdd_ctx* c) {
  const Net& A = c->A;
  const Buffers& B = c->B;
  const int rows = c->D.max_prompt - 1;
  int s = SDD_OK;
  if (A.dtype == SDD_BF16) {
    SDD_LAUNCH(c, CAT_GLUE, launch_embed_target<__nv_bfloat16>((const __nv_bfloat16*)A.wte, (const __nv_bfloat16*)A.wpe, B.tokens,
                                                               c->D.tok_stride, B.ctx_len, B.slot_ids, c->D.batch, c->D.gamma,
                                                               rows, TARGET_PREFILL, A.d, B.h, c->st, A.vocab, &B.rs->status));
    s = forward_causal<__nv_bfloat16>(c, A, c->ar_kv, B.ctx_len, TARGET_PREFILL, rows, false, nullptr, false, CAT_GEMM_Q,
                                      CAT_HEAD_Q, CAT_ATTN_Q);
  } else {
    SDD_LAUNCH(c, CAT_GLUE, launch_embed_target<float>((const float*)A.wte, (const float*)A.wpe, B.tokens, c->D.tok_stride,
                                                       B.ctx_len, B.slot_ids, c->D.batch, c->D.gamma, rows, TARGET_PREFILL, A.d,
                                                       B.h, c->st, A.vocab, &B.rs->status));
    s = forward_causal<float>(c, A, c->ar_kv, B.ctx_len, TARGET_PREFILL, rows, false, nullptr, false, CAT_GEMM_Q, CAT_HEAD_Q,
                              CAT_ATTN_Q);
  }
  return s;
}

static int enqueue_sps_round(sdd_ctx* c, int gamma, int32_t* out_ids, int32_t* n_out) {
  for (int j = 0; j < gamma; ++j)
    SDD_TRY(c->P.dtype == SDD_BF16 ? forward_ar_drafter<__nv_bfloat16>(c, gamma, j) : forward_ar_drafter<float>(c, gamma, j));
  return enqueue_verify_accept(c, gamma, out_ids, n_out);
}

// One round of standard speculative decoding with the attached autoregressive drafter: gamma_sps sequential drafter
// evaluations, then the same verification, acceptance and commit kernels as a SpecDiff round.
int32_t sdd_sps_step(sdd_ctx* c, int32_t gamma_sps, int32_t* out_ids, int32_t* n_out) {
  if (c == nullptr) return SDD_E_ARG;
  if (!c->has_ar || !c->sps_allowed || c->steps_done != -1) return SDD_E_STATE;
  if (gamma_sps < 1 || gamma_sps > c->D.gamma) return SDD_E_ARG;
  if (c->rounds >= (uint64_t)c->runahead)
    SDD_CUDA(cudaEventSynchronize(c->ev[(c->rounds - c->runahead) % c->ev.size()]));
  if (!c->use_graph || c->profiling) {
    SDD_TRY(enqueue_sps_round(c, gamma_sps, out_ids, n_out));
    return round_epilogue(c, gamma_sps + 1);
  }
  // keys of the other graphs: padded row counts (positive), 0 (autoregressive step), small negative (timing passes)
  const auto key = std::make_tuple(-(1 << 24) - gamma_sps, (void*)out_ids, (void*)n_out);
  auto it = c->graphs.find(key);
  if (it == c->graphs.end()) {
    const uint64_t l0 = c->launches;
    SDD_CUDA(cudaStreamBeginCapture(c->st, cudaStreamCaptureModeThreadLocal));
    const int s = enqueue_sps_round(c, gamma_sps, out_ids, n_out);
    cudaGraph_t g = nullptr;
    cudaError_t e = cudaStreamEndCapture(c->st, &g);
    if (s != SDD_OK) { if (g) cudaGraphDestroy(g); return s; }
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamEndCapture");
    sdd_ctx::GraphEntry ge;
    ge.exec = nullptr;
    ge.launches = c->launches - l0;
    c->launches = l0;
    e = cudaGraphInstantiate(&ge.exec, g, 0);
    cudaGraphDestroy(g);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGraphInstantiate");
    it = c->graphs.emplace(key, ge).first;
  }
  SDD_CUDA(cudaGraphLaunch(it->second.exec, c->st));
  c->launches += it->second.launches;
  return round_epilogue(c, gamma_sps + 1);
}

int32_t sdd_progress(sdd_ctx* c, uint64_t* rounds_done, int32_t* min_emitted) {
  if (c == nullptr) return SDD_E_ARG;
  const int Bn = c->D.batch;
  volatile int* m = c->mirror;
  for (int attempt = 0; attempt < 64; ++attempt) {
    // tail stamp, body, head stamp: the reverse of the commit kernel's write order (see choose_lcap)
    const int s1 = m[1 + 2 * Bn];
    std::atomic_thread_fence(std::memory_order_acquire);
    int mn = 0x7fffffff;
    for (int b = 0; b < Bn; ++b) { const int e = m[1 + Bn + b]; if (e < mn) mn = e; }
    std::atomic_thread_fence(std::memory_order_acquire);
    const int s0 = m[0];
    if (s0 == s1) {
      if (rounds_done) *rounds_done = (uint64_t)s1;
      if (min_emitted) *min_emitted = s1 == 0 ? 0 : mn;
      return SDD_OK;
    }
  }
  // a commit is being written right now: report the previous, consistent view conservatively
  if (rounds_done) *rounds_done = 0;
  if (min_emitted) *min_emitted = 0;
  return SDD_OK;
}

uint64_t sdd_accept_scratch_bytes(int32_t rows, int32_t gamma, int32_t V) {
  if (rows < 1 || gamma < 1 || V < 1) return 0;
  return (uint64_t)rows * (2ull * gamma + 1) * stats_chunks_for(V) * sizeof(float2);
}

int32_t sdd_accept_logits(const float* logits_p, const float* logits_q, const int32_t* draft_ids, int32_t rows,
                          int32_t gamma, int32_t V, float temp_p, float temp_q, uint64_t seed, uint64_t round,
                          int32_t* n_accept, int32_t* out_ids, float* accept_prob, void* scratch, void* stream) {
  if (!logits_p || !logits_q || !draft_ids || !n_accept || !out_ids || !accept_prob || !scratch) return SDD_E_ARG;
  if (rows < 1 || rows > 65535 || gamma < 1 || gamma > 256 || V < 2) return SDD_E_ARG;
  if (!(temp_p >= 0.f) || !(temp_q >= 0.f) || ((temp_p == 0.f) != (temp_q == 0.f))) return SDD_E_ARG;
  if (((uintptr_t)logits_p & 15u) || ((uintptr_t)logits_q & 15u) || ((uintptr_t)scratch & 15u)) return SDD_E_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const float itp = temp_p > 0.f ? 1.f / temp_p : 0.f, itq = temp_q > 0.f ? 1.f / temp_q : 0.f;
  float2* partial = (float2*)scratch;
  const long long rows_p = (long long)rows * (gamma + 1), rows_q = (long long)rows * gamma;
  const int chunks = stats_chunks_for(V);
  SDD_CUDA(launch_row_stats(logits_p, rows_p, logits_q, itp == 0.f ? 0 : rows_q, V, itp, itq, partial, st));
  SDD_CUDA(launch_accept(logits_p, logits_q, draft_ids, nullptr, nullptr, partial, chunks, partial + rows_p * chunks, chunks, rows, gamma, V, itp, itq,
                         make_key(seed), (uint32_t)round, nullptr, accept_prob, n_accept, nullptr, out_ids, st));
  return SDD_OK;
}

int32_t sdd_debug_gemm_bf16(const void* A, int64_t a_rows_capacity, const void* W, const float* bias, int32_t M, int32_t N,
                            int32_t K, int32_t epilogue, void* out, int32_t ldc, int32_t n_tile, int32_t use_tensor_cores,
                            int32_t* status_word, void* stream, const void* A_lo, void* out_lo) {
  if (!A || !W || !out || M < 1 || N < 1 || K < 8 || (K % 8) != 0 || epilogue < 0 || epilogue > 3) return SDD_E_ARG;
  if (a_rows_capacity < M || ldc < N) return SDD_E_ARG;
  if ((A_lo != nullptr || out_lo != nullptr) && !use_tensor_cores) return SDD_E_UNIMPL;
  if (out_lo != nullptr && epilogue > 1) return SDD_E_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (use_tensor_cores)
    SDD_CUDA(launch_gemm_tc((const __nv_bfloat16*)A, a_rows_capacity, (const __nv_bfloat16*)W, bias, M, N, K, epilogue, out,
                            ldc, n_tile, status_word, st, nullptr, (const __nv_bfloat16*)A_lo, out_lo));
  else
    SDD_CUDA(launch_gemm_simt<__nv_bfloat16>((const __nv_bfloat16*)A, K, (const __nv_bfloat16*)W, bias, M, N, K, epilogue,
                                             out, ldc, st));
  return SDD_OK;
}

int32_t sdd_debug_attention_bf16(const void* q, int64_t q_rows_total, int32_t q_ld, int32_t q_col0, const void* k,
                                 int64_t k_rows_total, int32_t k_ld, int32_t k_col0, int32_t k_rows_per_seq, const void* vt,
                                 int32_t vt_ld, void* out, int32_t ld_out, const int32_t* ctx_len, int32_t batch,
                                 int32_t n_head, int32_t gamma, int32_t mode, int32_t q_rows_per_seq, int32_t* status_word,
                                 void* stream) {
  if (!q || !k || !vt || !out || !ctx_len || batch < 1 || n_head < 1 || mode < 0 || mode > 2) return SDD_E_ARG;
  SDD_CUDA(launch_attn_tc((const __nv_bfloat16*)q, q_rows_total, q_ld, q_col0, (const __nv_bfloat16*)k, k_rows_total, k_ld,
                          k_col0, k_rows_per_seq, (const __nv_bfloat16*)vt, vt_ld, (__nv_bfloat16*)out, ld_out, ctx_len, batch,
                          n_head, n_head * 64, gamma, mode, q_rows_per_seq, status_word, (cudaStream_t)stream));
  return SDD_OK;
}

int32_t sdd_debug_wait_timeout(int64_t limit_cycles, int32_t* status_word, void* stream) {
  if (status_word == nullptr || limit_cycles < 1 || limit_cycles > 2000000000ll) return SDD_E_ARG;
  SDD_CUDA(launch_wait_timeout_probe((long long)limit_cycles, status_word, (cudaStream_t)stream));
  return SDD_OK;
}

int32_t sdd_tap(sdd_ctx* c, int32_t what, const void** dev_ptr, uint64_t* bytes) {
  if (c == nullptr || dev_ptr == nullptr || bytes == nullptr) return SDD_E_ARG;
  const Buffers& B = c->B;
  const uint64_t Bn = c->D.batch, G = c->D.gamma, V = c->D.V;
  switch (what) {
    case SDD_TAP_TOKENS: *dev_ptr = B.tokens; *bytes = Bn * c->D.tok_stride * 4; break;
    case SDD_TAP_CTX_LEN: *dev_ptr = B.ctx_len; *bytes = Bn * 4; break;
    case SDD_TAP_DRAFT_IDS: *dev_ptr = B.slot_ids; *bytes = Bn * G * 4; break;
    case SDD_TAP_STEP_LOGITS: *dev_ptr = B.step_logits; *bytes = Bn * G * V * 4; break;
    case SDD_TAP_Q_LOGITS: *dev_ptr = B.q_logits; *bytes = Bn * G * V * 4; break;
    case SDD_TAP_LOGQ: *dev_ptr = B.logq; *bytes = Bn * G * 4; break;
    case SDD_TAP_REVEAL_STEP: *dev_ptr = B.reveal_step; *bytes = Bn * G * 4; break;
    case SDD_TAP_LOGITS_P: *dev_ptr = B.logits_p; *bytes = Bn * (G + 1) * V * 4; break;
    case SDD_TAP_ACCEPT_PROB: *dev_ptr = B.accept_prob; *bytes = Bn * G * 4; break;
    case SDD_TAP_N_ACCEPT: *dev_ptr = B.n_accept; *bytes = Bn * 4; break;
    case SDD_TAP_EXTRA_TOKEN: *dev_ptr = B.extra_token; *bytes = Bn * 4; break;
    case SDD_TAP_N_EMITTED: *dev_ptr = B.n_emitted; *bytes = Bn * 4; break;
    case SDD_TAP_STATUS: *dev_ptr = &B.rs->status; *bytes = 4; break;
    case SDD_TAP_EVALS: *dev_ptr = &B.rs->evals_run; *bytes = 8; break;
    default: return SDD_E_ARG;
  }
  return SDD_OK;
}

int32_t sdd_counters(sdd_ctx* c, uint64_t* rounds, uint64_t* kernel_launches) {
  if (c == nullptr) return SDD_E_ARG;
  if (rounds) *rounds = c->rounds;
  if (kernel_launches) *kernel_launches = c->launches;
  return SDD_OK;
}

int32_t sdd_sync_status(sdd_ctx* c) {
  if (c == nullptr) return SDD_E_ARG;
  SDD_CUDA(cudaStreamSynchronize(c->st));
  int status = 0;
  SDD_CUDA(cudaMemcpy(&status, &c->B.rs->status, 4, cudaMemcpyDeviceToHost));
  if (status == DEV_OK) return SDD_OK;
  if (status == DEV_TIMEOUT) return SDD_E_TIMEOUT;
  return status == DEV_BAD_TOKEN ? SDD_E_INDEX : SDD_E_CTX_FULL;
}

int32_t sdd_profile_begin(sdd_ctx* c) {
  if (c == nullptr) return SDD_E_ARG;
  c->profiling = true;
  c->prof_used = 0;
  c->prof_cat.clear();
  return SDD_OK;
}

int32_t sdd_profile_end(sdd_ctx* c, double* ms_per_category, uint64_t* launches_per_category, int32_t n_categories) {
  if (c == nullptr || ms_per_category == nullptr || launches_per_category == nullptr) return SDD_E_ARG;
  if (n_categories < CAT_COUNT) return SDD_E_ARG;
  c->profiling = false;
  SDD_CUDA(cudaStreamSynchronize(c->st));
  for (int i = 0; i < n_categories; ++i) { ms_per_category[i] = 0.0; launches_per_category[i] = 0; }
  double empty_ms = 0.0;
  uint64_t empty_n = 0;
  for (size_t i = 0; i + 1 < c->prof_used + 1 && i / 2 < c->prof_cat.size(); i += 2) {
    float ms = 0.f;
    SDD_CUDA(cudaEventElapsedTime(&ms, c->prof_ev[i], c->prof_ev[i + 1]));
    const int cat = c->prof_cat[i / 2];
    if (cat == CAT_COUNT) { empty_ms += ms; empty_n += 1; continue; }
    ms_per_category[cat] += ms;
    launches_per_category[cat] += 1;
  }
  // subtract the cost of an empty event pair from every measured launch
  const double per_pair = empty_n ? empty_ms / (double)empty_n : 0.0;
  for (int i = 0; i < CAT_COUNT; ++i) {
    ms_per_category[i] -= per_pair * (double)launches_per_category[i];
    if (ms_per_category[i] < 0.0) ms_per_category[i] = 0.0;
  }
  c->prof_used = 0;
  c->prof_cat.clear();
  for (auto& k : c->prof_graphs) {
    auto it = c->graphs.find(k);
    if (it != c->graphs.end()) {
      if (it->second.exec) cudaGraphExecDestroy(it->second.exec);
      c->graphs.erase(it);
    }
  }
  c->prof_graphs.clear();
  return SDD_OK;
}

void sdd_destroy(sdd_ctx* c) {
  if (c == nullptr) return;
  for (auto e : c->prof_ev)
    if (e) cudaEventDestroy(e);
  for (auto& g : c->graphs)
    if (g.second.exec) cudaGraphExecDestroy(g.second.exec);
  for (auto e : c->ev)
    if (e) cudaEventDestroy(e);
  if (c->mirror) cudaFreeHost(c->mirror);
  delete c;
}

const char* sdd_strerror(int32_t s) {
  switch (s) {
    case SDD_OK: return "ok";
    case SDD_E_ARG: return "invalid argument";
    case SDD_E_SHAPE: return "unsupported or inconsistent model shape";
    case SDD_E_WORKSPACE: return "workspace too small or misaligned";
    case SDD_E_CTX_FULL: return "context would exceed the position table";
    case SDD_E_CUDA: return "CUDA call failed";
    case SDD_E_TIMEOUT: return "bounded device-side wait expired";
    case SDD_E_UNIMPL: return "not implemented";
    case SDD_E_STATE: return "call order violated";
    case SDD_E_INDEX: return "a token id or position outside its table was met on the device";
    default: return "unknown status";
  }
}

const char* sdd_last_cuda_error(void) { return g_cuda_err; }

}  // extern "C"
