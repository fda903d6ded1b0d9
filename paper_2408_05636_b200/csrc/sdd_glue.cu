// Small row-wise kernels around the GEMMs: embedding gather, LayerNorm, KV-cache append.
#include "sdd_kernels.h"

namespace sdd {

// ---------------------------------------------------------------------------------------------
// embeddings: h = wte[token] + wpe[position]
// drafter rows: sequence b owns rows b*L_cap .. b*L_cap + L_cap - 1; row i is context token i for
// i < c, draft slot i - c for c <= i < c + gamma, and zero padding beyond.
// ---------------------------------------------------------------------------------------------
constexpr int EMB_THREADS = 128;
constexpr int EMB_MAX_PER_THREAD = 16;   // d_model <= 2048
constexpr float EMB_LN_EPS = 1e-5f;      // the LayerNorm epsilon (same value as below)

// sum over the 128 threads of an embedding block (every thread gets the result)
__device__ __forceinline__ float emb_block_sum(float v, float* red) {
  v = warp_sum(v);
  __syncthreads();                       // red may still be read from the previous call
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  return (red[0] + red[1]) + (red[2] + red[3]);
}

// The embedding kernels also apply the first block's LayerNorm to the row they have just built (xn != nullptr), which
// saves that launch: x holds the thread's elements e = tid + 128 k of the row.
template <typename T>
__device__ __forceinline__ void emb_layernorm_store(const float (&x)[EMB_MAX_PER_THREAD], int d, const float* __restrict__ g,
                                                    const float* __restrict__ bta, T* __restrict__ xn_row) {
  __shared__ float red[4];
  float sum = 0.f;
#pragma unroll
  for (int k = 0; k < EMB_MAX_PER_THREAD; ++k) sum += (int)threadIdx.x + EMB_THREADS * k < d ? x[k] : 0.f;
  const float mu = emb_block_sum(sum, red) / (float)d;
  float var = 0.f;
#pragma unroll
  for (int k = 0; k < EMB_MAX_PER_THREAD; ++k) {
    const float cdev = (int)threadIdx.x + EMB_THREADS * k < d ? x[k] - mu : 0.f;
    var += cdev * cdev;
  }
  const float rstd = rsqrtf(emb_block_sum(var, red) / (float)d + EMB_LN_EPS);
#pragma unroll
  for (int k = 0; k < EMB_MAX_PER_THREAD; ++k) {
    const int e = (int)threadIdx.x + EMB_THREADS * k;
    if (e < d) xn_row[e] = from_f32<T>((x[k] - mu) * rstd * g[e] + bta[e]);
  }
}

template <typename T>
__global__ void __launch_bounds__(EMB_THREADS)
embed_drafter_kernel(const T* __restrict__ wte, const T* __restrict__ wpe, const int* __restrict__ tokens,
                     int tok_stride, const int* __restrict__ ctx_len, const int* __restrict__ slot_ids,
                     int gamma, int L_cap, int d, float* __restrict__ h, const int* __restrict__ skip,
                     const float* __restrict__ ln_g, const float* __restrict__ ln_b, T* __restrict__ xn, int vocab,
                     int* __restrict__ status) {
  pdl_launch_dependents();
  pdl_wait();
  if (skip != nullptr && *skip) return;
  const int i = blockIdx.x, b = blockIdx.y;
  const int c = ctx_len[b];
  const long long row = (long long)b * L_cap + i;
  float* __restrict__ dst = h + row * d;
  float x[EMB_MAX_PER_THREAD];
  // ids come from the caller's prompt: one outside [0, vocab] (vocab = [MASK]) must not index the table
  int tok = 0;
  if (i < c + gamma) {
    tok = i < c ? tokens[(long long)b * tok_stride + i] : slot_ids[(long long)b * gamma + (i - c)];
    if ((unsigned)tok > (unsigned)vocab) {
      if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, DEV_OK, DEV_BAD_TOKEN);
      tok = -1;
    }
  }
  if (i >= c + gamma || tok < 0) {           // padding row (or a bad id): zeros (its LayerNorm is the LayerNorm bias)
#pragma unroll
    for (int k = 0; k < EMB_MAX_PER_THREAD; ++k) x[k] = 0.f;
  } else {
    const T* __restrict__ te = wte + (long long)tok * d;
    const T* __restrict__ pe = wpe + (long long)i * d;
#pragma unroll
    for (int k = 0; k < EMB_MAX_PER_THREAD; ++k) {
      const int e = (int)threadIdx.x + EMB_THREADS * k;
      x[k] = e < d ? to_f32(te[e]) + to_f32(pe[e]) : 0.f;
    }
  }
#pragma unroll
  for (int k = 0; k < EMB_MAX_PER_THREAD; ++k) {
    const int e = (int)threadIdx.x + EMB_THREADS * k;
    if (e < d) dst[e] = x[k];
  }
  if (xn != nullptr) emb_layernorm_store<T>(x, d, ln_g, ln_b, xn + row * d);
}

// target rows: sequence b owns rows b*rows_per_seq ..; VERIFY: row j = [last context token, drafts] at
// position c-1+j; PREFILL: row j = context token j at position j (valid while j < c-1, else zero).
template <typename T>
__global__ void embed_target_kernel(const T* __restrict__ wte, const T* __restrict__ wpe, const int* __restrict__ tokens,
                                    int tok_stride, const int* __restrict__ ctx_len, const int* __restrict__ slot_ids,
                                    int gamma, int rows_per_seq, int mode, int d, float* __restrict__ h, int vocab,
                                    int* __restrict__ status) {
  pdl_launch_dependents();
  pdl_wait();
  const int j = blockIdx.x, b = blockIdx.y;
  const int c = ctx_len[b];
  float* __restrict__ dst = h + ((long long)b * rows_per_seq + j) * d;
  int tok, pos;
  bool pad = false;
  if (mode == TARGET_VERIFY) {
    pos = c - 1 + j;
    tok = j == 0 ? tokens[(long long)b * tok_stride + c - 1] : slot_ids[(long long)b * gamma + j - 1];
  } else {
    pos = j;
    pad = j >= c - 1;
    tok = pad ? 0 : tokens[(long long)b * tok_stride + j];
  }
  if (!pad && (unsigned)tok >= (unsigned)vocab) {   // a caller's id outside the table: zero row, reported through the status word
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, DEV_OK, DEV_BAD_TOKEN);
    pad = true;
  }
  if (pad) {
    for (int e = threadIdx.x; e < d; e += blockDim.x) dst[e] = 0.f;
    return;
  }
  const T* __restrict__ te = wte + (long long)tok * d;
  const T* __restrict__ pe = wpe + (long long)pos * d;
  for (int e = threadIdx.x; e < d; e += blockDim.x) dst[e] = to_f32(te[e]) + to_f32(pe[e]);
}

// Autoregressive drafter of a speculative-decoding round: row i of sequence b is position c + off - 1 + i, whose token
// is a context token (position < c) or a draft of this round (slot position - c).  Block (0, b) also publishes the
// evaluation's effective length c + off, which the other kernels of the evaluation take in place of ctx_len
// (their rows then sit at positions eff - 1 + i, the convention of a verification forward).
template <typename T>
__global__ void embed_ar_kernel(const T* __restrict__ wte, const T* __restrict__ wpe, const int* __restrict__ tokens,
                                int tok_stride, const int* __restrict__ ctx_len, const int* __restrict__ slot_ids,
                                int gamma, int rows_per_seq, int off, int d, float* __restrict__ h,
                                int* __restrict__ eff_len, int vocab, int* __restrict__ status) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = blockIdx.x, b = blockIdx.y;
  const int c = ctx_len[b];
  if (i == 0 && threadIdx.x == 0) eff_len[b] = c + off;
  const int pos = c + off - 1 + i;
  float* __restrict__ dst = h + ((long long)b * rows_per_seq + i) * d;
  if (pos < 0) {   // cannot happen for prompts of two or more tokens
    for (int e = threadIdx.x; e < d; e += blockDim.x) dst[e] = 0.f;
    return;
  }
  const int tok = pos < c ? tokens[(long long)b * tok_stride + pos] : slot_ids[(long long)b * gamma + pos - c];
  if ((unsigned)tok >= (unsigned)vocab) {    // an id outside the table: zero row, reported through the status word
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, DEV_OK, DEV_BAD_TOKEN);
    for (int e = threadIdx.x; e < d; e += blockDim.x) dst[e] = 0.f;
    return;
  }
  const T* __restrict__ te = wte + (long long)tok * d;
  const T* __restrict__ pe = wpe + (long long)pos * d;
  for (int e = threadIdx.x; e < d; e += blockDim.x) dst[e] = to_f32(te[e]) + to_f32(pe[e]);
}

// ---------------------------------------------------------------------------------------------
// LayerNorm (eps 1e-5): one warp per row, the row held in registers, mean then centred variance
// ---------------------------------------------------------------------------------------------
constexpr int LN_MAX_PER_LANE = 64;  // d_model <= 2048
constexpr float LN_EPS = 1e-5f;

template <typename T>
__device__ __forceinline__ void layernorm_row(const float* __restrict__ src, const float* __restrict__ g,
                                              const float* __restrict__ bta, T* __restrict__ dst, T* __restrict__ dst_lo,
                                              int d) {
  const int lane = threadIdx.x & 31;
  float x[LN_MAX_PER_LANE];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < LN_MAX_PER_LANE; ++i) {
    const int e = i * 32 + lane;
    x[i] = e < d ? src[e] : 0.f;
    sum += x[i];
  }
  const float mu = warp_sum(sum) / (float)d;
  float var = 0.f;
#pragma unroll
  for (int i = 0; i < LN_MAX_PER_LANE; ++i) {
    const int e = i * 32 + lane;
    const float c = e < d ? x[i] - mu : 0.f;
    var += c * c;
  }
  const float rstd = rsqrtf(warp_sum(var) / (float)d + LN_EPS);
#pragma unroll
  for (int i = 0; i < LN_MAX_PER_LANE; ++i) {
    const int e = i * 32 + lane;
    if (e < d) {
      const float y = (x[i] - mu) * rstd * g[e] + bta[e];
      const T hi = from_f32<T>(y);
      dst[e] = hi;
      if (dst_lo != nullptr) dst_lo[e] = from_f32<T>(y - to_f32<T>(hi));   // second half of a hi/lo pair
    }
  }
}

// Vector variant for the large forwards: every lane owns groups of four consecutive elements (16-byte loads of the
// fp32 row and of the gain / bias, 8- or 16-byte stores), NV groups per lane, d = 4 * 32 * NV at most and a multiple
// of 4; all pointers 16-byte aligned.
template <typename T>
__device__ __forceinline__ void store4(T* p, float a, float b, float c, float d);
template <>
__device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <>
__device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
}

template <typename T, int NV>
__global__ void __launch_bounds__(128)
layernorm_vec_kernel(const float* __restrict__ h, const float* __restrict__ g, const float* __restrict__ bta,
                     T* __restrict__ out, T* __restrict__ out_lo, long long rows, int d, const int* __restrict__ skip) {
  // gain and bias are weights (never written while the library runs): fetched before the wait for the kernel ahead
  const int lane = threadIdx.x & 31;
  float4 gg[NV], bb[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int e = (i * 32 + lane) * 4;
    if (e < d) { gg[i] = *reinterpret_cast<const float4*>(g + e); bb[i] = *reinterpret_cast<const float4*>(bta + e); }
    else { gg[i] = make_float4(0.f, 0.f, 0.f, 0.f); bb[i] = gg[i]; }
  }
  pdl_launch_dependents();
  pdl_wait();
  const long long row = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float* __restrict__ src = h + row * d;
  // the row's loads are issued before the skip flag is looked at, so that the two round trips overlap
  float4 x[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int e = (i * 32 + lane) * 4;
    x[i] = e < d ? *reinterpret_cast<const float4*>(src + e) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (skip != nullptr && *skip) return;
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) sum += (x[i].x + x[i].y) + (x[i].z + x[i].w);
  const float mu = warp_sum(sum) / (float)d;
  float var = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int e = (i * 32 + lane) * 4;
    if (e < d) {
      const float a = x[i].x - mu, b = x[i].y - mu, c = x[i].z - mu, dd = x[i].w - mu;
      var += (a * a + b * b) + (c * c + dd * dd);
    }
  }
  const float rstd = rsqrtf(warp_sum(var) / (float)d + LN_EPS);
  T* __restrict__ dst = out + row * d;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int e = (i * 32 + lane) * 4;
    if (e < d) {
      const float y0 = (x[i].x - mu) * rstd * gg[i].x + bb[i].x, y1 = (x[i].y - mu) * rstd * gg[i].y + bb[i].y;
      const float y2 = (x[i].z - mu) * rstd * gg[i].z + bb[i].z, y3 = (x[i].w - mu) * rstd * gg[i].w + bb[i].w;
      store4<T>(dst + e, y0, y1, y2, y3);
      if (out_lo != nullptr)   // second half of a hi/lo pair
        store4<T>(out_lo + row * d + e, y0 - to_f32<T>(from_f32<T>(y0)), y1 - to_f32<T>(from_f32<T>(y1)),
                  y2 - to_f32<T>(from_f32<T>(y2)), y3 - to_f32<T>(from_f32<T>(y3)));
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(128)
layernorm_kernel(const float* __restrict__ h, const float* __restrict__ g, const float* __restrict__ bta,
                 T* __restrict__ out, T* __restrict__ out_lo, long long rows, int d, const int* __restrict__ skip) {
  pdl_launch_dependents();
  pdl_wait();
  if (skip != nullptr && *skip) return;
  const long long row = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
  if (row >= rows) return;
  layernorm_row<T>(h + row * d, g, bta, out + row * d, out_lo != nullptr ? out_lo + row * d : nullptr, d);
}

template <typename T>
__global__ void __launch_bounds__(128)
layernorm_slots_kernel(const float* __restrict__ h, const float* __restrict__ g, const float* __restrict__ bta,
                       T* __restrict__ out, const int* __restrict__ ctx_len, int batch, int gamma, int L_cap, int d,
                       const int* __restrict__ skip) {
  pdl_launch_dependents();
  pdl_wait();
  if (skip != nullptr && *skip) return;
  const int r = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (r >= batch * gamma) return;
  const int b = r / gamma, j = r - b * gamma;
  layernorm_row<T>(h + ((long long)b * L_cap + ctx_len[b] + j) * d, g, bta, out + (long long)r * d, nullptr, d);
}

// ---------------------------------------------------------------------------------------------
// Slot-row gather: after the drafter's last attention only the gamma slot rows of every sequence feed the LM head, so
// the rest of that block runs on a compact copy: att_s[b*gamma + j] = att[b*L_cap + c_b + j], the same for h.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void gather_slots_kernel(const T* __restrict__ att, const float* __restrict__ h, const int* __restrict__ ctx_len,
                                    int gamma, int L_cap, int d, T* __restrict__ att_s, float* __restrict__ h_s,
                                    const int* __restrict__ skip) {
  pdl_launch_dependents();
  pdl_wait();
  if (skip != nullptr && *skip) return;
  const int j = blockIdx.x, b = blockIdx.y;
  const long long src = ((long long)b * L_cap + ctx_len[b] + j) * d, dst = ((long long)b * gamma + j) * d;
  for (int e = threadIdx.x; e < d; e += blockDim.x) {
    att_s[dst + e] = att[src + e];
    h_s[dst + e] = h[src + e];
  }
}

// ---------------------------------------------------------------------------------------------
// KV append: cache[b][pos][0] = K row, cache[b][pos][1] = V row
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void kv_append_kernel(const T* __restrict__ qkv, T* __restrict__ cache, const int* __restrict__ ctx_len,
                                 int rows_per_seq, int mode, int n_ctx, int d) {
  pdl_launch_dependents();
  pdl_wait();
  const int j = blockIdx.x, b = blockIdx.y;
  const int c = ctx_len[b];
  int pos;
  if (mode == TARGET_VERIFY) pos = c - 1 + j;
  else { if (j >= c - 1) return; pos = j; }
  if (pos >= n_ctx) return;
  const T* __restrict__ src = qkv + ((long long)b * rows_per_seq + j) * 3 * d + d;  // K then V, contiguous
  T* __restrict__ dst = cache + ((long long)b * n_ctx + pos) * 2 * d;
  for (int e = threadIdx.x; e < 2 * d; e += blockDim.x) dst[e] = src[e];
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
template <typename T>
cudaError_t launch_embed_drafter(const T* wte, const T* wpe, const int* tokens, int tok_stride, const int* ctx_len,
                                 const int* slot_ids, int batch, int gamma, int L_cap, int d, float* h, cudaStream_t st,
                                 const int* skip, const float* ln_g, const float* ln_b, T* xn, int vocab, int* status) {
  if (d > EMB_THREADS * EMB_MAX_PER_THREAD) return cudaErrorInvalidValue;
  launch_k(embed_drafter_kernel<T>, dim3(L_cap, batch), dim3(EMB_THREADS), 0, st, wte, wpe, tokens, tok_stride, ctx_len, slot_ids,
           gamma, L_cap, d, h, skip, ln_g, ln_b, xn, vocab, status);
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_embed_target(const T* wte, const T* wpe, const int* tokens, int tok_stride, const int* ctx_len,
                                const int* slot_ids, int batch, int gamma, int rows_per_seq, int mode, int d, float* h,
                                cudaStream_t st, int vocab, int* status) {
  if (rows_per_seq <= 0) return cudaSuccess;
  launch_k(embed_target_kernel<T>, dim3(dim3(rows_per_seq, batch)), dim3(128), 0, st, wte, wpe, tokens, tok_stride, ctx_len, slot_ids, gamma,
                                                                    rows_per_seq, mode, d, h, vocab, status);
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_embed_ar(const T* wte, const T* wpe, const int* tokens, int tok_stride, const int* ctx_len,
                            const int* slot_ids, int batch, int gamma, int rows_per_seq, int off, int d, float* h,
                            int* eff_len, cudaStream_t st, int vocab, int* status) {
  launch_k(embed_ar_kernel<T>, dim3(rows_per_seq, batch), dim3(128), 0, st, wte, wpe, tokens, tok_stride, ctx_len, slot_ids,
           gamma, rows_per_seq, off, d, h, eff_len, vocab, status);
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_layernorm(const float* h, const float* g, const float* b, T* out, long long rows, int d,
                             cudaStream_t st, T* out_lo, const int* skip) {
  if (rows <= 0) return cudaSuccess;
  if (d > LN_MAX_PER_LANE * 32) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)((rows + 3) / 4));
  const uintptr_t al = reinterpret_cast<uintptr_t>(h) | reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(b) |
                       reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(out_lo);
  if ((d & 3) == 0 && (al & 15u) == 0) {
    if (d <= 1024) launch_k(layernorm_vec_kernel<T, 8>, grid, dim3(128), 0, st, h, g, b, out, out_lo, rows, d, skip);
    else launch_k(layernorm_vec_kernel<T, 16>, grid, dim3(128), 0, st, h, g, b, out, out_lo, rows, d, skip);
  } else {
    launch_k(layernorm_kernel<T>, grid, dim3(128), 0, st, h, g, b, out, out_lo, rows, d, skip);
  }
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_layernorm_slots(const float* h, const float* g, const float* b, T* out, const int* ctx_len, int batch,
                                   int gamma, int L_cap, int d, cudaStream_t st, const int* skip) {
  if (d > LN_MAX_PER_LANE * 32) return cudaErrorInvalidValue;
  launch_k(layernorm_slots_kernel<T>, dim3((batch * gamma + 3) / 4), dim3(128), 0, st, h, g, b, out, ctx_len, batch, gamma, L_cap, d, skip);
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_gather_slots(const T* att, const float* h, const int* ctx_len, int batch, int gamma, int L_cap, int d,
                                T* att_s, float* h_s, cudaStream_t st, const int* skip) {
  launch_k(gather_slots_kernel<T>, dim3(gamma, batch), dim3(128), 0, st, att, h, ctx_len, gamma, L_cap, d, att_s, h_s, skip);
  return cudaGetLastError();
}
template <typename T>
cudaError_t launch_kv_append(const T* qkv, T* cache, const int* ctx_len, int batch, int rows_per_seq, int mode, int n_ctx,
                             int d, cudaStream_t st) {
  if (rows_per_seq <= 0) return cudaSuccess;
  launch_k(kv_append_kernel<T>, dim3(dim3(rows_per_seq, batch)), dim3(128), 0, st, qkv, cache, ctx_len, rows_per_seq, mode, n_ctx, d);
  return cudaGetLastError();
}

#define SDD_INSTANTIATE_GLUE(T)                                                                                          \
  template cudaError_t launch_embed_drafter<T>(const T*, const T*, const int*, int, const int*, const int*, int, int,   \
                                               int, int, float*, cudaStream_t, const int*, const float*, const float*,  \
                                               T*, int, int*);                                                          \
  template cudaError_t launch_embed_target<T>(const T*, const T*, const int*, int, const int*, const int*, int, int,    \
                                              int, int, int, float*, cudaStream_t, int, int*);                          \
  template cudaError_t launch_embed_ar<T>(const T*, const T*, const int*, int, const int*, const int*, int, int, int,   \
                                          int, int, float*, int*, cudaStream_t, int, int*);                             \
  template cudaError_t launch_layernorm<T>(const float*, const float*, const float*, T*, long long, int, cudaStream_t, \
                                           T*, const int*);                                                                         \
  template cudaError_t launch_layernorm_slots<T>(const float*, const float*, const float*, T*, const int*, int, int,    \
                                                 int, int, cudaStream_t, const int*);                                   \
  template cudaError_t launch_gather_slots<T>(const T*, const float*, const int*, int, int, int, int, T*, float*,       \
                                              cudaStream_t, const int*);                                                \
  template cudaError_t launch_kv_append<T>(const T*, T*, const int*, int, int, int, int, int, cudaStream_t);
SDD_INSTANTIATE_GLUE(float)
SDD_INSTANTIATE_GLUE(__nv_bfloat16)

}  // namespace sdd
