// Attention kernels of the two networks (CUDA-core version: one warp per (query row, head)).
//   bidirectional (drafter): softmax(Q K^T / sqrt(d_head)) V over all rows of the sequence, no mask
//   cached causal (target) : row at position p attends to KV-cache positions 0..p
// Scores are computed one key per lane, the online soft-max state is per warp, and P V is accumulated
// with one output dimension (pair) per lane.
#include "sdd_kernels.h"

namespace sdd {

template <typename T, int DH>
__device__ __forceinline__ void attn_one_query(const T* __restrict__ q, const T* __restrict__ kbase,
                                               const T* __restrict__ vbase, long long kv_stride, int n_keys,
                                               T* __restrict__ out) {
  constexpr int PER_LANE = DH / 32;
  const int lane = threadIdx.x & 31;
  const float scale = rsqrtf((float)DH);
  float qr[DH];
#pragma unroll
  for (int e = 0; e < DH; ++e) qr[e] = to_f32(q[e]) * scale;
  float m = -INFINITY, l = 0.f;
  float acc[PER_LANE];
#pragma unroll
  for (int e = 0; e < PER_LANE; ++e) acc[e] = 0.f;
  for (int k0 = 0; k0 < n_keys; k0 += 32) {
    const int i = k0 + lane;
    float s = -INFINITY;
    if (i < n_keys) {
      const T* __restrict__ kr = kbase + (long long)i * kv_stride;
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < DH; ++e) dot = fmaf(qr[e], to_f32(kr[e]), dot);
      s = dot;
    }
    const float m_new = fmaxf(m, warp_max(s));
    const float corr = expf(m - m_new);           // m = -inf on the first block: exp(-inf) = 0
    const float p = i < n_keys ? expf(s - m_new) : 0.f;
    l = l * corr + warp_sum(p);
#pragma unroll
    for (int e = 0; e < PER_LANE; ++e) acc[e] *= corr;
    const int nk = min(32, n_keys - k0);
    for (int kk = 0; kk < nk; ++kk) {
      const float pk = __shfl_sync(0xffffffffu, p, kk);
      const T* __restrict__ vr = vbase + (long long)(k0 + kk) * kv_stride;
#pragma unroll
      for (int e = 0; e < PER_LANE; ++e) acc[e] = fmaf(pk, to_f32(vr[e * 32 + lane]), acc[e]);
    }
    m = m_new;
  }
  const float inv = 1.f / l;
#pragma unroll
  for (int e = 0; e < PER_LANE; ++e) out[e * 32 + lane] = from_f32<T>(acc[e] * inv);
}

template <typename T, int DH>
__global__ void __launch_bounds__(128)
attn_bidir_kernel(const T* __restrict__ qkv, T* __restrict__ out, const int* __restrict__ ctx_len, int gamma, int L_cap,
                  int n_head, const int* __restrict__ skip) {
  pdl_launch_dependents();
  pdl_wait();
  if (skip != nullptr && *skip) return;
  const int i = blockIdx.x * 4 + (threadIdx.x >> 5), h = blockIdx.y, b = blockIdx.z;
  if (i >= L_cap) return;
  const int d = n_head * DH;
  const int L = ctx_len[b] + gamma;
  const long long row0 = (long long)b * L_cap;
  T* __restrict__ o = out + (row0 + i) * d + h * DH;
  if (i >= L) {   // padding row: keep it finite
    for (int e = threadIdx.x & 31; e < DH; e += 32) o[e] = from_f32<T>(0.f);
    return;
  }
  const T* __restrict__ base = qkv + row0 * 3 * d + h * DH;
  attn_one_query<T, DH>(base + (long long)i * 3 * d, base + d, base + 2 * d, 3ll * d, L, o);
}

template <typename T, int DH>
__global__ void __launch_bounds__(128)
attn_cached_kernel(const T* __restrict__ qkv, const T* __restrict__ cache, T* __restrict__ out,
                   const int* __restrict__ ctx_len, int rows_per_seq, int mode, int n_ctx, int n_head) {
  pdl_launch_dependents();
  pdl_wait();
  const int j = blockIdx.x * 4 + (threadIdx.x >> 5), h = blockIdx.y, b = blockIdx.z;
  if (j >= rows_per_seq) return;
  const int d = n_head * DH;
  const int c = ctx_len[b];
  const long long row = (long long)b * rows_per_seq + j;
  T* __restrict__ o = out + row * d + h * DH;
  int pos;
  bool valid;
  if (mode == TARGET_VERIFY) { pos = c - 1 + j; valid = pos < n_ctx; }
  else { pos = j; valid = j < c - 1; }
  if (!valid) {
    for (int e = threadIdx.x & 31; e < DH; e += 32) o[e] = from_f32<T>(0.f);
    return;
  }
  const T* __restrict__ kb = cache + (long long)b * n_ctx * 2 * d + h * DH;
  attn_one_query<T, DH>(qkv + row * 3 * d + h * DH, kb, kb + d, 2ll * d, pos + 1, o);
}

template <typename T>
cudaError_t launch_attn_bidir(const T* qkv, T* out, const int* ctx_len, int batch, int gamma, int L_cap, int n_head,
                              int d_head, cudaStream_t st, const int* skip) {
  dim3 grid((L_cap + 3) / 4, n_head, batch);
  if (d_head == 64) launch_k(attn_bidir_kernel<T, 64>, dim3(grid), dim3(128), 0, st, qkv, out, ctx_len, gamma, L_cap, n_head, skip);
  else if (d_head == 32) launch_k(attn_bidir_kernel<T, 32>, dim3(grid), dim3(128), 0, st, qkv, out, ctx_len, gamma, L_cap, n_head, skip);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

template <typename T>
cudaError_t launch_attn_cached(const T* qkv, const T* cache, T* out, const int* ctx_len, int batch, int rows_per_seq,
                               int mode, int n_ctx, int n_head, int d_head, cudaStream_t st) {
  if (rows_per_seq <= 0) return cudaSuccess;
  dim3 grid((rows_per_seq + 3) / 4, n_head, batch);
  if (d_head == 64)
    launch_k(attn_cached_kernel<T, 64>, dim3(grid), dim3(128), 0, st, qkv, cache, out, ctx_len, rows_per_seq, mode, n_ctx, n_head);
  else if (d_head == 32)
    launch_k(attn_cached_kernel<T, 32>, dim3(grid), dim3(128), 0, st, qkv, cache, out, ctx_len, rows_per_seq, mode, n_ctx, n_head);
  else return cudaErrorInvalidValue;
  return cudaGetLastError();
}

#define SDD_INSTANTIATE_ATTN(T)                                                                                  \
  template cudaError_t launch_attn_bidir<T>(const T*, T*, const int*, int, int, int, int, int, cudaStream_t,   \
                                            const int*);                                                       \
  template cudaError_t launch_attn_cached<T>(const T*, const T*, T*, const int*, int, int, int, int, int, int, \
                                             cudaStream_t);
SDD_INSTANTIATE_ATTN(float)
SDD_INSTANTIATE_ATTN(__nv_bfloat16)

}  // namespace sdd
