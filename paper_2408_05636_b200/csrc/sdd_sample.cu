// Memory-bound vocabulary kernels of a SpecDiff round (Algorithm 1):
//   row_stats_kernel      soft-max statistics (max, sum exp) of logit rows, one streaming pass
//   unmask_sample_kernel  one denoising step's reveal test + Gumbel-max draw + stored q row
//   accept_kernel         u <= min(1, p/q) scan, residual norm(max(0, p - q)) or bonus draw
//   commit_kernel         append the emitted tokens to each sequence
#include <cooperative_groups.h>

#include "sdd_kernels.h"

namespace sdd {

// ---------------------------------------------------------------------------------------------
// row statistics
//
// grid = logical rows * chunks per row (chunk index fastest).  A logical row is V floats starting
// at element row * V of a 16-byte aligned buffer, so a row start is in general only 4-byte aligned.
// Each CTA covers STATS_CHUNK elements of the 16-byte-aligned span that contains the row, with
// float4 loads; elements outside the row are masked, and a float4 that is not wholly inside the
// row is read by scalars.  Output: one (max, sum exp(z - max)) pair per (row, chunk) with
// z = x * inv_tau; in greedy mode (inv_tau == 0) the pair is (max x, index of the first maximum
// as an int bit pattern).
// ---------------------------------------------------------------------------------------------
constexpr int STATS_THREADS = 256;
constexpr int STATS_VEC_PER_THREAD = 8;
constexpr int STATS_CHUNK = STATS_THREADS * STATS_VEC_PER_THREAD * 4;  // 8192 elements

__host__ __device__ inline int stats_chunks(int V) { return (V + 3 + STATS_CHUNK - 1) / STATS_CHUNK; }

template <bool GREEDY>
__global__ void __launch_bounds__(STATS_THREADS)
row_stats_kernel(const float* __restrict__ buf_a, long long rows_a, const float* __restrict__ buf_b, long long rows_b,
                 int V, int chunks, float inv_tau_a, float inv_tau_b, float2* __restrict__ partial) {
  pdl_launch_dependents();
  pdl_wait();
  const long long row = blockIdx.x / chunks;
  const int chunk = blockIdx.x - (int)(row * chunks);
  const bool is_a = row < rows_a;
  const float* __restrict__ buf = is_a ? buf_a : buf_b;
  const long long lrow = is_a ? row : row - rows_a;
  const float inv_tau = is_a ? inv_tau_a : inv_tau_b;
  const long long r0 = lrow * V, r1 = r0 + V;           // flat element range of this row
  const long long base = (r0 & ~3ll) + (long long)chunk * STATS_CHUNK;

  float x[STATS_VEC_PER_THREAD][4];
#pragma unroll
  for (int i = 0; i < STATS_VEC_PER_THREAD; ++i) {
    const long long e = base + ((long long)i * STATS_THREADS + threadIdx.x) * 4;
    if (e >= r0 && e + 3 < r1) {
      const float4 v = __ldcs(reinterpret_cast<const float4*>(buf + e));
      x[i][0] = v.x; x[i][1] = v.y; x[i][2] = v.z; x[i][3] = v.w;
    } else {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const long long ec = e + c;
        x[i][c] = (ec >= r0 && ec < r1) ? __ldcs(buf + ec) : -INFINITY;
      }
    }
  }

  __shared__ float s_m[STATS_THREADS / 32];
  __shared__ float s_s[STATS_THREADS / 32];
  __shared__ int s_i[STATS_THREADS / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  if (GREEDY) {
    ArgMax a;
    a.s = -INFINITY;
    a.i = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < STATS_VEC_PER_THREAD; ++i) {
      const long long e = base + ((long long)i * STATS_THREADS + threadIdx.x) * 4;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        ArgMax b;
        b.s = x[i][c];
        b.i = (int)(e + c - r0);
        if (b.s > -INFINITY) a = argmax_better(a, b);
      }
    }
    a = warp_argmax(a);
    if (lane == 0) { s_m[warp] = a.s; s_i[warp] = a.i; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < STATS_THREADS / 32; ++w) {
        ArgMax b;
        b.s = s_m[w]; b.i = s_i[w];
        a = argmax_better(a, b);
      }
      partial[blockIdx.x] = make_float2(a.s, __int_as_float(a.i));
    }
    return;
  }

  float m = -INFINITY;
#pragma unroll
  for (int i = 0; i < STATS_VEC_PER_THREAD; ++i)
#pragma unroll
    for (int c = 0; c < 4; ++c) m = fmaxf(m, x[i][c]);
  m = warp_max(m);
  if (lane == 0) s_m[warp] = m;
  __syncthreads();
  m = s_m[0];
#pragma unroll
  for (int w = 1; w < STATS_THREADS / 32; ++w) m = fmaxf(m, s_m[w]);
  // m is the chunk maximum of x (or -inf for an empty chunk); accumulate sum exp((x - m) * inv_tau)
  float s = 0.f;
  if (m > -INFINITY) {
    const float k = inv_tau * 1.4426950408889634f;
    const float mk = m * k;
#pragma unroll
    for (int i = 0; i < STATS_VEC_PER_THREAD; ++i)
#pragma unroll
      for (int c = 0; c < 4; ++c) s += exp2f(fmaf(x[i][c], k, -mk));
  }
  s = warp_sum(s);
  if (lane == 0) s_s[warp] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < STATS_THREADS / 32; ++w) s += s_s[w];
    partial[blockIdx.x] = make_float2(m * inv_tau, s);
  }
}

// Merge of the per-chunk pairs of one row by a group of `tpr` consecutive lanes (a power of two up to 32; `sub` = the
// lane's index in its group): the log-sum-exp of z, valid in every lane of the group.  All 32 lanes of the warp call it
// together (the shuffles are warp-wide); a group whose row does not exist passes valid = false.
__device__ __forceinline__ float merge_partials(const float2* __restrict__ p, int chunks, int tpr, int sub, bool valid) {
  float m = -INFINITY;
  if (valid)
    for (int c = sub; c < chunks; c += tpr) m = fmaxf(m, p[c].x);
  for (int o = tpr >> 1; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float s = 0.f;
  if (valid)
    for (int c = sub; c < chunks; c += tpr) {
      const float2 v = p[c];
      if (v.x > -INFINITY) s += v.y * expf(v.x - m);
    }
  for (int o = tpr >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  return m + logf(s);
}
__device__ __forceinline__ int merge_partials_argmax(const float2* __restrict__ p, int chunks, int tpr, int sub, bool valid) {
  ArgMax a;
  a.s = -INFINITY;
  a.i = 0x7fffffff;
  if (valid)
    for (int c = sub; c < chunks; c += tpr) {
      ArgMax b;
      b.s = p[c].x;
      b.i = __float_as_int(p[c].y);
      if (b.s > -INFINITY) a = argmax_better(a, b);
    }
  for (int o = tpr >> 1; o > 0; o >>= 1) {
    ArgMax b;
    b.s = __shfl_xor_sync(0xffffffffu, a.s, o);
    b.i = __shfl_xor_sync(0xffffffffu, a.i, o);
    a = argmax_better(a, b);
  }
  return a.i;
}
// lanes that share a row when rows of `chunks` pairs are merged: one thread per row for the few pairs that
// row_stats_kernel leaves (all rows of a sequence are then merged at once), a warp per row for the hundreds that the
// LM head's epilogue leaves
__device__ __forceinline__ int merge_group_size(int chunks) { return chunks <= 8 ? 1 : 32; }

// block-wide arg-max; result valid in thread 0
template <int THREADS>
__device__ __forceinline__ ArgMax block_argmax(ArgMax a, float* s_val, int* s_idx) {
  a = warp_argmax(a);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { s_val[warp] = a.s; s_idx[warp] = a.i; }
  __syncthreads();
  if (warp == 0) {
    ArgMax b;
    b.s = lane < THREADS / 32 ? s_val[lane] : -INFINITY;
    b.i = lane < THREADS / 32 ? s_idx[lane] : 0x7fffffff;
    a = warp_argmax(b);
  }
  return a;
}

// block-wide log-sum-exp of an online accumulator; result valid in every thread
template <int THREADS>
__device__ __forceinline__ float block_lse(MaxSum ms, float* s_m, float* s_s, float* s_out) {
  ms = warp_maxsum(ms);
  if ((threadIdx.x & 31) == 0) { s_m[threadIdx.x >> 5] = ms.m; s_s[threadIdx.x >> 5] = ms.s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    MaxSum t;
    t.m = s_m[0]; t.s = s_s[0];
    for (int w = 1; w < THREADS / 32; ++w) {
      MaxSum o;
      o.m = s_m[w]; o.s = s_s[w];
      t = maxsum_merge(t, o);
    }
    *s_out = t.m + logf(t.s);
  }
  __syncthreads();
  return *s_out;
}

__device__ __forceinline__ void maxsum_push(MaxSum& ms, float z) {
  if (z > ms.m) { ms.s = ms.s * __expf(ms.m - z) + 1.f; ms.m = z; }
  else ms.s += __expf(z - ms.m);
}

// ---------------------------------------------------------------------------------------------
// The two vocabulary-wide draws below give one logit row to a thread-block cluster of VC CTAs: each
// CTA scans an interleaved 1/VC of the row, reduces inside the block, publishes its partial result
// in its own shared memory, and after a cluster barrier the partials are merged through distributed
// shared memory.  A single CTA per row would leave the row's latency chain (Philox, two logs, the
// scan over 50 k entries) on one SM.
// ---------------------------------------------------------------------------------------------
namespace cg = cooperative_groups;
constexpr int VC = 8;

struct RowPartial {
  float arg_s; int arg_i;      // Gumbel arg-max of this CTA's share
  float fb_s; int fb_i;        // fall-back arg-max (draw from p itself)
  float m, s;                  // online soft-max pair of this CTA's share
};

__device__ __forceinline__ ArgMax cluster_merge_argmax(cg::cluster_group& cl, RowPartial* mine, bool fallback) {
  ArgMax a;
  a.s = -INFINITY;
  a.i = 0x7fffffff;
  for (int r = 0; r < VC; ++r) {
    const RowPartial* o = cl.map_shared_rank(mine, r);
    ArgMax b;
    b.s = fallback ? o->fb_s : o->arg_s;
    b.i = fallback ? o->fb_i : o->arg_i;
    a = argmax_better(a, b);
  }
  return a;
}
__device__ __forceinline__ float cluster_merge_lse(cg::cluster_group& cl, RowPartial* mine) {
  MaxSum t;
  t.m = -INFINITY;
  t.s = 0.f;
  for (int r = 0; r < VC; ++r) {
    const RowPartial* o = cl.map_shared_rank(mine, r);
    MaxSum b;
    b.m = o->m; b.s = o->s;
    t = maxsum_merge(t, b);
  }
  return t.m + logf(t.s);
}

// block-wide online soft-max pair; result valid in thread 0
template <int THREADS>
__device__ __forceinline__ MaxSum block_maxsum(MaxSum ms, float* s_m, float* s_s) {
  ms = warp_maxsum(ms);
  if ((threadIdx.x & 31) == 0) { s_m[threadIdx.x >> 5] = ms.m; s_s[threadIdx.x >> 5] = ms.s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < THREADS / 32; ++w) {
      MaxSum o;
      o.m = s_m[w]; o.s = s_s[w];
      ms = maxsum_merge(ms, o);
    }
  }
  return ms;
}

// ---------------------------------------------------------------------------------------------
// denoising step k: reveal test, Gumbel-max draw, stored q row     grid = (VC * gamma, batch), cluster VC
// ---------------------------------------------------------------------------------------------
constexpr int SAMPLE_THREADS = 512;

// returns true in every CTA of a cluster whose slot was revealed by this step
// Gumbel-max draw of one slot by the cluster that owns it: x = argmax_v (z_v + G_v), z = src * inv_tau_q (arg-max of
// src when greedy); the row z is stored to dst, log q(x) = z_x - logsumexp(z) to *logq_out and logsumexp(z) to
// *lseq_out.  `mark` goes to
// *reveal_out (the denoising step, or the evaluation index of an autoregressive drafter).
__device__ __forceinline__ void draw_slot(const float* __restrict__ src, float* __restrict__ dst, int* __restrict__ slot_out,
                                          float* __restrict__ logq_out, float* __restrict__ lseq_out,
                                          int* __restrict__ reveal_out, int j, int b, int V,
                                          int mark, float inv_tau_q, PhiloxKey key, uint32_t rnd, int* __restrict__ status) {
  cg::cluster_group cl = cg::this_cluster();
  const int rank = (int)cl.block_rank();
  const bool greedy = inv_tau_q == 0.f;
  const uint32_t c3 = rng_c3(RNG_DRAFT, 0u, (uint32_t)b);

  MaxSum ms;
  ms.m = -INFINITY;
  ms.s = 0.f;
  ArgMax best;
  best.s = -INFINITY;
  best.i = 0x7fffffff;
  const int nblk = (V + 3) >> 2;
  for (int blk = rank * SAMPLE_THREADS + threadIdx.x; blk < nblk; blk += VC * SAMPLE_THREADS) {
    uint4 w = make_uint4(0, 0, 0, 0);
    if (!greedy) w = philox4x32_10((uint32_t)blk, (uint32_t)j, rnd, c3, key);
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int v = blk * 4 + c;
      if (v < V) {
        const float x = src[v];
        const float z = greedy ? x : x * inv_tau_q;
        dst[v] = z;
        ArgMax cand;
        cand.i = v;
        cand.s = greedy ? z : z + gumbel_from_uniform(word_to_uniform(ww[c]));
        best = argmax_better(best, cand);
        if (!greedy) maxsum_push(ms, z);
      }
    }
  }
  __shared__ float s_val[SAMPLE_THREADS / 32];
  __shared__ int s_idx[SAMPLE_THREADS / 32];
  __shared__ float s_m[SAMPLE_THREADS / 32], s_s[SAMPLE_THREADS / 32];
  __shared__ RowPartial part;
  best = block_argmax<SAMPLE_THREADS>(best, s_val, s_idx);
  ms = block_maxsum<SAMPLE_THREADS>(ms, s_m, s_s);
  if (threadIdx.x == 0) {
    part.arg_s = best.s; part.arg_i = best.i; part.m = ms.m; part.s = ms.s;
  }
  cl.sync();
  if (rank == 0 && threadIdx.x == 0) {
    ArgMax win = cluster_merge_argmax(cl, &part, false);
    const float lse = greedy ? 0.f : cluster_merge_lse(cl, &part);
    if ((unsigned)win.i >= (unsigned)V) {   // no entry compared greater than -inf: the logits are not numbers
      win.i = 0;
      if (status != nullptr) atomicCAS(status, DEV_OK, DEV_BAD_TOKEN);
    }
    *slot_out = win.i;
    *logq_out = greedy ? 0.f : src[win.i] * inv_tau_q - lse;
    *lseq_out = lse;               // the stored row's log-sum-exp: the residual draw of the acceptance step needs it
    *reveal_out = mark;
  }
  cl.sync();   // partials stay alive until rank 0 has read them
}

__device__ __forceinline__ bool unmask_sample_row(const float* __restrict__ step_logits,  // [B, gamma, V]
                     int* __restrict__ slot_ids,             // [B, gamma]  (V = masked)
                     float* __restrict__ q_logits,           // [B, gamma, V]
                     float* __restrict__ logq,               // [B, gamma]
                     float* __restrict__ lseq,               // [B, gamma]
                     int* __restrict__ reveal_step,          // [B, gamma]
                     int gamma, int V, int k, float inv_tau_q, PhiloxKey key, RoundState* __restrict__ rs) {
  const int j = blockIdx.x / VC, b = blockIdx.y;
  const uint32_t rnd = rs->round;
  const long long row = (long long)b * gamma + j;
  // every CTA of the cluster takes the same decision from the same inputs, before anyone writes the slot
  if (slot_ids[row] != V) return false;  // already revealed: carried over unchanged
  // reveal with probability 1/k: u = m * 2^-24 with m odd, so u < 1/k  <=>  m * k < 2^24 (exact, k <= 255)
  const uint32_t wu = philox4x32_10(0u, (uint32_t)j, rnd, rng_c3(RNG_UNMASK, (uint32_t)k, (uint32_t)b), key).x;
  const uint32_t m_odd = ((wu >> 9) << 1) | 1u;
  if (!(m_odd * (uint32_t)k < (1u << 24))) return false;
  draw_slot(step_logits + row * V, q_logits + row * V, slot_ids + row, logq + row, lseq + row, reveal_step + row, j, b, V, k,
            inv_tau_q, key, rnd, &rs->status);
  return true;
}


// The last CTA of the grid to finish publishes whether this step revealed anything at all: if not, the next drafter
// evaluation would see the same input and reproduce the logits it already has, so its kernels are told to return
// at once (the paper's "ddpm cache" strategy: a step without change costs no network evaluation).
__global__ void __cluster_dims__(VC, 1, 1) __launch_bounds__(SAMPLE_THREADS)
unmask_sample_kernel(const float* __restrict__ step_logits, int* __restrict__ slot_ids, float* __restrict__ q_logits,
                     float* __restrict__ logq, float* __restrict__ lseq, int* __restrict__ reveal_step, int gamma, int V, int k,
                     float inv_tau_q, PhiloxKey key, RoundState* __restrict__ rs, int cache_skip) {
  pdl_launch_dependents();
  pdl_wait();
  const bool revealed = unmask_sample_row(step_logits, slot_ids, q_logits, logq, lseq, reveal_step, gamma, V, k, inv_tau_q, key, rs);
  if (threadIdx.x == 0) {
    if (revealed && (blockIdx.x % VC) == 0) atomicAdd(&rs->revealed, 1u);
    __threadfence();
    const uint32_t t = atomicAdd(&rs->ticket, 1u);
    if (t == gridDim.x * gridDim.y - 1) {
      __threadfence();
      const uint32_t n = atomicExch(&rs->revealed, 0u);
      // the flag as it stood during this step tells whether the step's drafter evaluation ran
      if (rs->skip_forward) rs->evals_skipped += 1; else rs->evals_run += 1;
      rs->skip_forward = (cache_skip && n == 0u) ? 1 : 0;
      rs->ticket = 0u;
    }
  }
}

// Draw of slot j by an autoregressive drafter (standard speculative decoding): the logits are the last of the
// `rows_per_seq` rows the evaluation produced for each sequence; the slot is always written.  grid = (VC, batch).
__global__ void __cluster_dims__(VC, 1, 1) __launch_bounds__(SAMPLE_THREADS)
ar_sample_kernel(const float* __restrict__ logits, int rows_per_seq, int* __restrict__ slot_ids, float* __restrict__ q_logits,
                 float* __restrict__ logq, float* __restrict__ lseq, int* __restrict__ reveal_step, int gamma, int j, int V,
                 float inv_tau_q, PhiloxKey key, RoundState* __restrict__ rs) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.y;
  const long long row = (long long)b * gamma + j;
  draw_slot(logits + ((long long)b * rows_per_seq + rows_per_seq - 1) * V, q_logits + row * V, slot_ids + row, logq + row,
            lseq + row, reveal_step + row, j, b, V, gamma - j, inv_tau_q, key, rs->round, &rs->status);
}

// ---------------------------------------------------------------------------------------------
// acceptance scan + extra token                                  grid = (VC * rows), cluster VC per row
//
// logits_p [rows, gamma+1, V]; q rows [rows, gamma, V] hold z_q = l * inv_tau_q_rows (inv_tau_q_rows
// = 1 when the rows were stored already divided by the temperature).  log q(x) and the q rows' log-sum-exp come
// either from `logq_in` / `lseq_in` (round pipeline: stored by the draw) or from the q-row partial statistics
// (stand-alone call).  A draft id outside [0, V) is never used as an index: its row counts as rejected, the
// sequence's n_accept becomes -1 (out_ids all -1) and, in the round pipeline, the status word DEV_BAD_TOKEN.
// ---------------------------------------------------------------------------------------------
constexpr int ACCEPT_THREADS = 256;

// four CTAs per SM (64 registers): the stand-alone call's 8 x rows CTAs then fit in one wave for 64 rows
__global__ void __cluster_dims__(VC, 1, 1) __launch_bounds__(ACCEPT_THREADS, 4)
accept_kernel(const float* __restrict__ logits_p, const float* __restrict__ q_rows, const int* __restrict__ draft_ids,
              const float* __restrict__ logq_in, const float* __restrict__ lseq_in, const float2* __restrict__ partial_p,
              int chunks, const float2* __restrict__ partial_q, int chunks_q, int gamma, int V, float inv_tau_p,
              float inv_tau_q_rows, PhiloxKey key, uint32_t rnd_arg, RoundState* __restrict__ rs,
              float* __restrict__ accept_prob, int* __restrict__ n_accept, int* __restrict__ extra_token,
              int* __restrict__ out_ids) {
  pdl_launch_dependents();
  pdl_wait();
  cg::cluster_group cl = cg::this_cluster();
  const int rank = (int)cl.block_rank();
  const int b = blockIdx.x / VC;
  const uint32_t rnd = rs != nullptr ? rs->round : rnd_arg;
  const bool greedy = inv_tau_p == 0.f;
  extern __shared__ float s_dyn[];           // [gamma+1] lse_p (or arg-max bits), [gamma] lse_q
  float* s_lsep = s_dyn;
  float* s_lseq = s_dyn + gamma + 1;
  __shared__ int s_n, s_bad;
  __shared__ int s_rej[ACCEPT_THREADS / 32];
  __shared__ float s_val[ACCEPT_THREADS / 32];
  __shared__ int s_idx[ACCEPT_THREADS / 32];
  __shared__ RowPartial part;

  if (threadIdx.x == 0) s_bad = 0;
  const float2* pp = partial_p + (long long)b * (gamma + 1) * chunks;
  // the rows' pairs are merged by groups of lanes sized to the number of pairs (7 from row_stats_kernel: a thread per
  // row; 393 from the LM head's epilogue: a warp per row)
  {
    const int tpr = merge_group_size(chunks), sub = (int)threadIdx.x % tpr, par = ACCEPT_THREADS / tpr;
    for (int j0 = 0; j0 <= gamma; j0 += par) {
      const int j = j0 + (int)threadIdx.x / tpr;
      const bool valid = j <= gamma;
      const float2* row = pp + (long long)(valid ? j : 0) * chunks;
      const float v = greedy ? __int_as_float(merge_partials_argmax(row, chunks, tpr, sub, valid))
                             : merge_partials(row, chunks, tpr, sub, valid);
      if (valid && sub == 0) s_lsep[j] = v;
    }
  }
  if (partial_q != nullptr && !greedy) {
    const float2* pq = partial_q + (long long)b * gamma * chunks_q;
    const int tpr = merge_group_size(chunks_q), sub = (int)threadIdx.x % tpr, par = ACCEPT_THREADS / tpr;
    for (int j0 = 0; j0 < gamma; j0 += par) {
      const int j = j0 + (int)threadIdx.x / tpr;
      const bool valid = j < gamma;
      const float v = merge_partials(pq + (long long)(valid ? j : 0) * chunks_q, chunks_q, tpr, sub, valid);
      if (valid && sub == 0) s_lseq[j] = v;
    }
  }
  __syncthreads();

  // first rejected position, computed identically by every CTA of the cluster (gamma <= ACCEPT_THREADS)
  int rej = gamma;
  if ((int)threadIdx.x < gamma) {
    const int j = threadIdx.x;
    const int x = draft_ids[(long long)b * gamma + j];
    float ratio;
    if ((unsigned)x >= (unsigned)V) {
      ratio = 0.f;
      s_bad = 1;
    } else if (greedy) {
      ratio = (x == __float_as_int(s_lsep[j])) ? 1.f : 0.f;
    } else {
      const float logp = logits_p[((long long)b * (gamma + 1) + j) * V + x] * inv_tau_p - s_lsep[j];
      const float lq = logq_in != nullptr ? logq_in[(long long)b * gamma + j]
                                          : q_rows[((long long)b * gamma + j) * V + x] * inv_tau_q_rows - s_lseq[j];
      ratio = expf(fminf(0.f, logp - lq));
    }
    const float u = scalar_uniform(key, RNG_ACCEPT, rnd, 0u, (uint32_t)j, (uint32_t)b);
    if (rank == 0) accept_prob[(long long)b * gamma + j] = ratio;
    if (!(u <= ratio)) rej = j;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) rej = min(rej, __shfl_xor_sync(0xffffffffu, rej, o));
  if ((threadIdx.x & 31) == 0) s_rej[threadIdx.x >> 5] = rej;
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = gamma;
    for (int w = 0; w < ACCEPT_THREADS / 32; ++w) n = min(n, s_rej[w]);
    s_n = n;
  }
  __syncthreads();
  const int n = s_n;

  // extra token: residual of row n (n < gamma) or the bonus draw from row gamma
  const float* __restrict__ prow = logits_p + ((long long)b * (gamma + 1) + n) * V;
  const bool resid = n < gamma;
  ArgMax best, fallback;
  best.s = -INFINITY;
  best.i = 0x7fffffff;
  fallback = best;
  if (!greedy) {
    const float* __restrict__ qrow = q_rows + ((long long)b * gamma + (resid ? n : 0)) * V;
    const float lsep = s_lsep[n];
    float lseq = 0.f;
    if (resid) {
      // stand-alone call: from the q rows' chunk statistics; round pipeline: stored by the draw of slot n
      lseq = partial_q != nullptr ? s_lseq[n] : lseq_in[(long long)b * gamma + n];
    }
    const uint32_t c3 = rng_c3(resid ? RNG_RESID : RNG_BONUS, 0u, (uint32_t)b);
    const int nblk = (V + 3) >> 2;
    // two blocks of four entries per iteration, with all loads of the iteration issued before any arithmetic
    constexpr int UNR = 2;
    for (int blk0 = rank * ACCEPT_THREADS + threadIdx.x; blk0 < nblk; blk0 += UNR * VC * ACCEPT_THREADS) {
      float xp[UNR][4], xq[UNR][4];
#pragma unroll
      for (int u = 0; u < UNR; ++u) {
        const int blk = blk0 + u * VC * ACCEPT_THREADS;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int v = blk * 4 + c;
          const bool in = blk < nblk && v < V;
          xp[u][c] = in ? __ldg(prow + v) : 0.f;
          xq[u][c] = (in && resid) ? __ldg(qrow + v) : 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < UNR; ++u) {
        const int blk = blk0 + u * VC * ACCEPT_THREADS;
        if (blk >= nblk) break;
        const uint4 w = philox4x32_10((uint32_t)blk, (uint32_t)n, rnd, c3, key);
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int v = blk * 4 + c;
          if (v < V) {
            const float g = gumbel_from_uniform(word_to_uniform(ww[c]));
            const float zp = xp[u][c] * inv_tau_p - lsep;   // log p_v
            ArgMax cand;
            cand.i = v;
            cand.s = zp + g;
            if (resid) {
              fallback = argmax_better(fallback, cand);    // a draw from p itself, if max(0, p - q) == 0 everywhere
              const float zq = xq[u][c] * inv_tau_q_rows - lseq;
              const float wv = __expf(zp) - __expf(zq);
              if (wv > 0.f) {
                cand.s = __logf(wv) + g;
                best = argmax_better(best, cand);
              }
            } else {
              best = argmax_better(best, cand);
            }
          }
        }
      }
    }
    best = block_argmax<ACCEPT_THREADS>(best, s_val, s_idx);
    __syncthreads();
    fallback = block_argmax<ACCEPT_THREADS>(fallback, s_val, s_idx);
  }
  if (threadIdx.x == 0) {
    part.arg_s = best.s; part.arg_i = best.i; part.fb_s = fallback.s; part.fb_i = fallback.i;
  }
  cl.sync();
  if (rank == 0 && threadIdx.x == 0) {
    int t;
    if (greedy) {
      t = __float_as_int(s_lsep[n]);   // arg-max of the target row, in both branches
    } else {
      ArgMax win = cluster_merge_argmax(cl, &part, false);
      if (win.i == 0x7fffffff) win = cluster_merge_argmax(cl, &part, true);
      t = win.i;
    }
    bool bad = s_bad != 0;
    if ((unsigned)t >= (unsigned)V) {   // no entry compared greater than -inf: the logits are not numbers
      t = 0;
      bad = true;
    }
    if (bad && rs != nullptr) atomicCAS(&rs->status, DEV_OK, DEV_BAD_TOKEN);
    n_accept[b] = bad ? -1 : n;
    if (extra_token != nullptr) extra_token[b] = t;
    if (out_ids != nullptr) {
      for (int j = 0; j <= gamma; ++j)
        out_ids[(long long)b * (gamma + 1) + j] = bad ? -1 : (j < n ? draft_ids[(long long)b * gamma + j] : (j == n ? t : -1));
    }
  }
  cl.sync();   // partials stay alive until rank 0 has read them
}

// ---------------------------------------------------------------------------------------------
// commit: append x_1..x_n, t to every sequence (Algorithm 1, "Return"), truncated to max_new
// one block; host_mirror (mapped pinned memory, may be null) = [stamp, ctx_len[B], n_emitted[B], stamp]
// ---------------------------------------------------------------------------------------------
__global__ void commit_kernel(int* __restrict__ tokens, int tok_stride, int* __restrict__ ctx_len,
                              int* __restrict__ n_emitted, const int* __restrict__ slot_ids,
                              const int* __restrict__ n_accept, const int* __restrict__ extra_token, int batch, int gamma,
                              int max_new, RoundState* rs, int* __restrict__ out_ids, int* __restrict__ n_out,
                              volatile int* host_mirror) {
  pdl_launch_dependents();
  pdl_wait();
  const uint32_t stamp = rs->round + 1u;
  if (host_mirror != nullptr && threadIdx.x == 0) {
    host_mirror[0] = (int)stamp;
    __threadfence_system();
  }
  __syncthreads();
  for (int b = threadIdx.x; b < batch; b += blockDim.x) {
    const int c = ctx_len[b], e = n_emitted[b];
    const int n = n_accept[b];
    int emit = n + 1;
    if (emit > max_new - e) emit = max_new - e;
    if (emit < 0) emit = 0;
    if (c + emit > tok_stride) {  // cannot happen when the host checked n_ctx; never write out of bounds
      emit = tok_stride - c;
      atomicCAS(&rs->status, DEV_OK, DEV_BAD_INDEX);
    }
    for (int j = 0; j < emit; ++j) {
      const int t = j < n ? slot_ids[(long long)b * gamma + j] : extra_token[b];
      tokens[(long long)b * tok_stride + c + j] = t;
    }
    if (out_ids != nullptr)
      for (int j = 0; j <= gamma; ++j)
        out_ids[(long long)b * (gamma + 1) + j] =
            j < emit ? (j < n ? slot_ids[(long long)b * gamma + j] : extra_token[b]) : -1;
    if (n_out != nullptr) n_out[b] = emit;
    ctx_len[b] = c + emit;
    n_emitted[b] = e + emit;
    if (host_mirror != nullptr) {
      host_mirror[1 + b] = c + emit;
      host_mirror[1 + batch + b] = e + emit;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    rs->round = stamp;
    if (host_mirror != nullptr) {
      __threadfence_system();
      host_mirror[1 + 2 * batch] = (int)stamp;
    }
  }
}

__global__ void reset_slots_kernel(int* __restrict__ slot_ids, int* __restrict__ reveal_step, int n, int mask_id,
                                   RoundState* __restrict__ rs) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0) { rs->skip_forward = 0; rs->revealed = 0u; rs->ticket = 0u; }   // a round's first evaluation always runs
  if (i < n) {
    slot_ids[i] = mask_id;
    reveal_step[i] = 0;
  }
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
int stats_chunks_for(int V) { return stats_chunks(V); }

cudaError_t launch_row_stats(const float* a, long long rows_a, const float* b, long long rows_b, int V, float inv_tau_a,
                             float inv_tau_b, float2* partial, cudaStream_t st) {
  const long long rows = rows_a + rows_b;
  if (rows <= 0) return cudaSuccess;
  const int chunks = stats_chunks(V);
  if (rows * chunks > 0x7fffffffll) return cudaErrorInvalidValue;
  const unsigned grid = (unsigned)(rows * chunks);
  if (inv_tau_a == 0.f)
    launch_k(row_stats_kernel<true>, dim3(grid), dim3(STATS_THREADS), 0, st, a, rows_a, b, rows_b, V, chunks, inv_tau_a, inv_tau_b, partial);
  else
    launch_k(row_stats_kernel<false>, dim3(grid), dim3(STATS_THREADS), 0, st, a, rows_a, b, rows_b, V, chunks, inv_tau_a, inv_tau_b, partial);
  return cudaGetLastError();
}

cudaError_t launch_unmask_sample(const float* step_logits, int* slot_ids, float* q_logits, float* logq, float* lseq,
                                 int* reveal_step, int batch, int gamma, int V, int k, float inv_tau_q, PhiloxKey key,
                                 RoundState* rs, int cache_skip, cudaStream_t st) {
  dim3 grid(VC * gamma, batch);
  launch_k(unmask_sample_kernel, dim3(grid), dim3(SAMPLE_THREADS), 0, st, step_logits, slot_ids, q_logits, logq, lseq, reveal_step, gamma,
           V, k, inv_tau_q, key, rs, cache_skip);
  return cudaGetLastError();
}

cudaError_t launch_ar_sample(const float* logits, int rows_per_seq, int* slot_ids, float* q_logits, float* logq, float* lseq,
                             int* reveal_step, int batch, int gamma, int j, int V, float inv_tau_q, PhiloxKey key,
                             RoundState* rs, cudaStream_t st) {
  launch_k(ar_sample_kernel, dim3(VC, batch), dim3(SAMPLE_THREADS), 0, st, logits, rows_per_seq, slot_ids, q_logits, logq, lseq,
           reveal_step, gamma, j, V, inv_tau_q, key, rs);
  return cudaGetLastError();
}

cudaError_t launch_accept(const float* logits_p, const float* q_rows, const int* draft_ids, const float* logq_in,
                          const float* lseq_in, const float2* partial_p, int chunks_p, const float2* partial_q, int chunks_q,
                          int rows, int gamma, int V,
                          float inv_tau_p, float inv_tau_q_rows, PhiloxKey key, uint32_t rnd, RoundState* rs, float* accept_prob,
                          int* n_accept, int* extra_token, int* out_ids, cudaStream_t st) {
  const size_t smem = (size_t)(2 * gamma + 1) * sizeof(float);
  launch_k(accept_kernel, dim3(VC * rows), dim3(ACCEPT_THREADS), smem, st, logits_p, q_rows, draft_ids, logq_in, lseq_in, partial_p,
                                                    chunks_p, partial_q, chunks_q, gamma, V, inv_tau_p, inv_tau_q_rows, key, rnd, rs,
                                                    accept_prob, n_accept, extra_token, out_ids);
  return cudaGetLastError();
}

cudaError_t launch_commit(int* tokens, int tok_stride, int* ctx_len, int* n_emitted, const int* slot_ids,
                          const int* n_accept, const int* extra_token, int batch, int gamma, int max_new, RoundState* rs,
                          int* out_ids, int* n_out, volatile int* host_mirror, cudaStream_t st) {
  launch_k(commit_kernel, dim3(1), dim3(256), 0, st, tokens, tok_stride, ctx_len, n_emitted, slot_ids, n_accept, extra_token, batch, gamma,
                                   max_new, rs, out_ids, n_out, host_mirror);
  return cudaGetLastError();
}

cudaError_t launch_reset_slots(int* slot_ids, int* reveal_step, int n, int mask_id, RoundState* rs, cudaStream_t st) {
  launch_k(reset_slots_kernel, dim3((n + 255) / 256), dim3(256), 0, st, slot_ids, reveal_step, n, mask_id, rs);
  return cudaGetLastError();
}

}  // namespace sdd
