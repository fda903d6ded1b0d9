// bf16 tensor-core GEMM for sm_100a:  C[M, N] = A[M, K] * W[N, K]^T  (fp32 accumulate) with fused epilogues.
//
// One CTA computes one 128 x BN accumulator tile that lives in tensor memory (TMEM).  Operand tiles
// (128 x 64 and BN x 64 bf16, K-major, 128-byte swizzle) are brought into a shared-memory ring by TMA
// (cp.async.bulk.tensor, one elected producer thread), consumed by tcgen05.mma issued from one elected
// thread, and the finished accumulator is read back with tcgen05.ld by four epilogue warps.
//
// Three kernels share the epilogues: gemm_tc_kernel (one tile per CTA; single-wave grids, K splits),
// gemm_tc_persist_kernel (one CTA per SM walks over tiles with two accumulators; many-tile grids and the LM heads) and
// gemm_tc_pair_kernel (two CTAs of a cluster share a 256 x 256 tile, tcgen05 cta_group::2; the largest GEMMs).  The host
// picks the kernel, the tile width and the K splits (launch_gemm_tc).
//
// Orientation.  NORMAL: MMA-M axis = activation rows, MMA-N axis = output features (large-M GEMMs of
// the drafter).  SWAP: MMA-M axis = output features (rows of W), MMA-N axis = tokens -- for the target's
// verification forward, where only gamma+1 tokens exist and the kernel is a weight-streaming pass; the
// epilogue then writes the transposed tile so that consecutive lanes write consecutive features.
//
// HILO: the activation operand may come as two bf16 tensors, hi = bf16(x) and lo = bf16(x - hi), and the kernel
// accumulates W x hi + W x lo into the same TMEM tile (16 significant bits of the activations instead of 8).  The
// target network's MLP and LM-head products use it: their logits are compared against an fp64 oracle, and the
// rounding of the activations to bf16 is the largest error term of a 48-layer forward.
//
// Every wait on an mbarrier is bounded: when the limit passes the thread raises the CTA's abort flag and
// the device status word, all roles leave their loops, the producer waits (bounded) for the copies it
// still has in flight, TMEM is freed and the CTA returns.
#include <cudaTypedefs.h>

#include <cstdlib>

#include <map>
#include <mutex>
#include <tuple>

#include "sdd_kernels.h"
#include "sdd_tc.cuh"

namespace sdd {

namespace tc {

constexpr int BM = 128;          // MMA M
constexpr int BK = 64;           // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int THREADS = 192;     // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, warps 2-5: epilogue

// tensor maps of the epilogue's TMA stores: the output matrix and (fused QKV of the drafter) the transposed V tensor
struct alignas(64) OutMaps { CUtensorMap out, vt; };

// one stage = A tile + B tile (+ the lo tile of the activation operand: the A side unless SWAP)
template <int BN, bool SWAP, bool HILO>
constexpr int stage_bytes() { return BM * BK * 2 + BN * BK * 2 + (HILO ? (SWAP ? BN : BM) * BK * 2 : 0); }
// shared-memory ring depth.  DEEP (grids of at most one wave): as deep as one CTA per SM allows (about 200 KB), so
// that a short K loop has all of its tiles in flight at once.  Otherwise (multi-wave grids): half of that, so that two
// CTAs share an SM and one's epilogue and prologue overlap the other's main loop.
template <int BN, bool SWAP, bool HILO, bool DEEP>
constexpr int ring_stages() {
  constexpr int s = ((DEEP ? 200 : 100) * 1024) / stage_bytes<BN, SWAP, HILO>();
  return s > 8 ? 8 : (s < 2 ? 2 : s);
}
template <int BN, bool SWAP, bool HILO, bool DEEP>
constexpr int smem_bytes() {
  return ring_stages<BN, SWAP, HILO, DEEP>() * stage_bytes<BN, SWAP, HILO>() + 1024 /*alignment slack*/ + 256 /*barriers*/ +
         1024 /*bias*/;
}

// ---------------------------------------------------------------------------------------------
// epilogues (shared by the one-tile and the persistent kernel); called by the four epilogue warps, q = TMEM lane
// quarter of the calling warp, tmem_acc = first column of the tile's accumulator
// ---------------------------------------------------------------------------------------------
// A group of four epilogue warps (128 threads, one TMEM lane quarter each) and the 32-column chunks it drains.  The
// one-CTA kernels have one group for the whole tile with two staging buffers; the pair kernel has two groups, each
// with half of the tile's chunks, one staging buffer and named barriers of its own.
struct EpiGroup {
  int c_begin, c_end;    // chunks [c_begin, c_end) of the tile; c_begin is even
  int nbuf;              // staging buffers of 16 KB at stage_generic: 1 or 2
  int bar_id;            // named barrier of the group's 128 threads
  int first_tid;         // first thread of the group; it issues the group's TMA stores
};
template <int BN>
__device__ __forceinline__ EpiGroup whole_tile_group() { return EpiGroup{0, BN / 32, 2, 2, 64}; }

// the group copies the bias values of its chunks to shared memory (zero past column N or without a bias)
__device__ __forceinline__ void stage_bias(float* bias_s, const float* __restrict__ bias, int n0, int rows_b, const EpiGroup& eg) {
  for (int c = eg.c_begin * 32 + (int)threadIdx.x - eg.first_tid; c < eg.c_end * 32; c += 128)
    bias_s[c] = (bias != nullptr && n0 + c < rows_b) ? bias[n0 + c] : 0.f;
  named_bar_sync(eg.bar_id, 128);
}
template <int BN>
__device__ __forceinline__ void stage_bias(float* bias_s, const float* __restrict__ bias, int n0, int rows_b) {
  stage_bias(bias_s, bias, n0, rows_b, whole_tile_group<BN>());
}

template <int BN>
__device__ __forceinline__ void epilogue_tma(uint32_t tmem_acc, int m0, int n0, int q, int lane, int epi,
                                             const float* bias_s, const CUtensorMap* map_out,
                                             uint8_t* stage_generic, uint32_t stage_u32, int& n_store,
                                             const EpiGroup eg = whole_tile_group<BN>()) {
  // Output through shared memory and TMA: every thread writes its row's 128-byte piece of the tile into a
  // staging buffer (128-byte swizzle, so that the 32 rows of a warp spread over all banks), one thread issues a
  // tile store (bf16 outputs) or an add-reduce (fp32 residual stream; also correct under K splits).
  // bias_s: the tile's BN bias values in shared memory (zeros where there is no bias or no column).
  const int rl = q * 32 + lane;               // row inside the tile
  const int sw = rl & 7;
  const bool is_issuer = (int)threadIdx.x == eg.first_tid;
  const bool f32 = epi == EPI_RESIDUAL;
  // groups of four chunks or more (256-column tiles) fetch two chunks from TMEM per wait (c_begin is even): half as many
  // exposed round trips to tensor memory; narrower tiles measured slower that way and keep one load per wait
  uint32_t vv[2][32];
  const int step = eg.c_end - eg.c_begin >= 4 ? 2 : 1;
  #pragma unroll 1
  for (int cc0 = eg.c_begin; cc0 < eg.c_end; cc0 += step) {
    const bool two = step == 2 && cc0 + 1 < eg.c_end;
    tmem_ld32_issue(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc0 * 32), vv[0]);
    if (two) tmem_ld32_issue(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)((cc0 + 1) * 32), vv[1]);
    tmem_ld_wait(vv[0], vv[1]);
#pragma unroll
   for (int half = 0; half < 2; ++half) {
    if (half == 1 && !two) break;
    const int cc = cc0 + half;
    const uint32_t (&v)[32] = vv[half];
    const int c0 = n0 + cc * 32;
    // fp32: one 32-column chunk fills a 128-byte row; bf16: two chunks do
    const int buf = eg.nbuf == 1 ? 0 : (f32 ? (cc & 1) : ((cc >> 1) & 1));
    const bool first_of_buf = f32 || (cc & 1) == 0;
    const bool last_of_buf = f32 || (cc & 1) == 1 || cc == eg.c_end - 1;
    if (first_of_buf) {
      // the store that last used this buffer has read it
      if (is_issuer && n_store >= eg.nbuf) { if (eg.nbuf == 1) tma_wait_group_read<0>(); else tma_wait_group_read<1>(); }
      named_bar_sync(eg.bar_id, 128);
    }
    uint8_t* row = stage_generic + buf * (128 * 128) + rl * 128;
    if (f32) {
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        float4 x;
        x.x = __uint_as_float(v[g * 4 + 0]) + bias_s[cc * 32 + g * 4 + 0];
        x.y = __uint_as_float(v[g * 4 + 1]) + bias_s[cc * 32 + g * 4 + 1];
        x.z = __uint_as_float(v[g * 4 + 2]) + bias_s[cc * 32 + g * 4 + 2];
        x.w = __uint_as_float(v[g * 4 + 3]) + bias_s[cc * 32 + g * 4 + 3];
        *reinterpret_cast<float4*>(row + ((g ^ sw) << 4)) = x;
      }
    } else {
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        uint32_t pk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int j0 = g * 8 + 2 * e;
          float x0 = __uint_as_float(v[j0]) + bias_s[cc * 32 + j0];
          float x1 = __uint_as_float(v[j0 + 1]) + bias_s[cc * 32 + j0 + 1];
          if (epi == EPI_GELU) { x0 = gelu_tanh_fast(x0); x1 = gelu_tanh_fast(x1); }
          __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
          pk[e] = *reinterpret_cast<uint32_t*>(&h2);
        }
        const int chunk = (cc & 1) * 4 + g;
        *reinterpret_cast<uint4*>(row + ((chunk ^ sw) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      }
    }
    if (last_of_buf) {
      fence_async_smem();
      named_bar_sync(eg.bar_id, 128);
      if (is_issuer) {
        const uint32_t src = stage_u32 + buf * (128 * 128);
        if (f32) tma_reduce_add_2d(map_out, src, c0, m0);
        else tma_store_2d(map_out, src, n0 + (cc & ~1) * 32, m0);
        tma_commit_group();
      }
      ++n_store;
    }
   }
  }
}

// V tiles of the drafter's fused-QKV GEMM: the tile is written transposed ([feature][position]) into the staging
// buffers -- 64 features x 128 positions per buffer, as two 128-byte-swizzled boxes of 64 positions -- and leaves
// through two TMA tile stores per buffer.  The 128 rows of the tile are 128 consecutive positions of one sequence.
// vt_row0: row of the tile's first feature in the V^T tensor; pos0: position of the tile's first row.
template <int BN>
__device__ __forceinline__ void epilogue_vt(uint32_t tmem_acc, int q, int lane, const float* bias_s,
                                            const CUtensorMap* map_vt, uint8_t* stage_generic, uint32_t stage_u32,
                                            int& n_store, int vt_row0, int pos0,
                                            const EpiGroup eg = whole_tile_group<BN>()) {
  const int rl = q * 32 + lane;               // row inside the tile = position offset
  const bool is_issuer = (int)threadIdx.x == eg.first_tid;
  const int pl = rl & 63;
  const uint32_t box_off = (uint32_t)(rl >> 6) * (64 * 128);       // positions 64..127 fill the second box
  const uint32_t in_row = (uint32_t)(pl & 7) * 2u;
  const uint32_t pchunk = (uint32_t)(pl >> 3);
#pragma unroll 1
  for (int cc = eg.c_begin; cc < eg.c_end; ++cc) {
    uint32_t v[32];
    tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 32), v);
    const int buf = eg.nbuf == 1 ? 0 : ((cc >> 1) & 1);
    const bool first_of_buf = (cc & 1) == 0;
    const bool last_of_buf = (cc & 1) == 1 || cc == eg.c_end - 1;
    if (first_of_buf) {
      // the stores that last used this buffer have read it
      if (is_issuer && n_store >= eg.nbuf) { if (eg.nbuf == 1) tma_wait_group_read<0>(); else tma_wait_group_read<1>(); }
      named_bar_sync(eg.bar_id, 128);
    }
    uint8_t* bp = stage_generic + buf * (128 * 128) + box_off;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const int jj = (cc & 1) * 32 + j;        // feature row inside the buffer
      const float x = __uint_as_float(v[j]) + bias_s[cc * 32 + j];
      *reinterpret_cast<__nv_bfloat16*>(bp + jj * 128 + ((pchunk ^ (uint32_t)(jj & 7)) << 4) + in_row) = __float2bfloat16_rn(x);
    }
    if (last_of_buf) {
      fence_async_smem();
      named_bar_sync(eg.bar_id, 128);
      if (is_issuer) {
        const uint32_t src = stage_u32 + buf * (128 * 128);
        const int y = vt_row0 + (cc & ~1) * 32;
        tma_store_2d(map_vt, src, pos0, y);
        tma_store_2d(map_vt, src + 64 * 128, pos0 + 64, y);
        tma_commit_group();
      }
      ++n_store;
    }
  }
}

template <int BN, bool SWAP, bool ROLL = false>
__device__ __forceinline__ void epilogue_manual(uint32_t tmem_acc, int m0, int n0, int q, int lane, int rows_a, int rows_b,
                                                int epi, const float* __restrict__ bias, void* __restrict__ out,
                                                void* __restrict__ out_lo, int ldc, bool split, const QkvDst& qd,
                                                int c_begin = 0, int c_end = BN / 32) {
  const int r = m0 + q * 32 + lane;          // index along the A operand's rows
  const bool r_ok = r < rows_a;
#pragma unroll 1
  for (int cc = c_begin; cc < c_end; ++cc) {
    uint32_t v[32];
    tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 32), v);
    const int c0 = n0 + cc * 32;             // index along the B operand's rows
    if (!SWAP) {
      // out[r][c]: r = token row, c = feature
      if (r_ok && epi == EPI_QKV && c0 >= 2 * qd.d) {
        // V chunk of token row r: transposed store, consecutive lanes = consecutive positions
        const int sb = r / qd.rows_per_seq, si = r - sb * qd.rows_per_seq;
        const int cl = qd.ctx_len[sb];
        const int pos = qd.mode == 1 ? cl - 1 + si : si;
        if ((qd.mode != 2 || si < cl - 1) && pos < qd.vt_ld) {
          __nv_bfloat16* vt = qd.vt_dst + ((long long)sb * qd.d + (c0 - 2 * qd.d)) * qd.vt_ld + pos;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c0 + j < rows_b) vt[(long long)j * qd.vt_ld] = __float2bfloat16_rn(__uint_as_float(v[j]) + (bias ? bias[c0 + j] : 0.f));
        }
      } else if (r_ok && epi == EPI_QKV && c0 >= qd.d && qd.k_dst != nullptr) {
        const int sb = r / qd.rows_per_seq, si = r - sb * qd.rows_per_seq;
        const int cl = qd.ctx_len[sb];
        const int pos = qd.mode == 1 ? cl - 1 + si : si;
        if ((qd.mode != 2 || si < cl - 1) && pos < qd.k_seq_rows) {
          __nv_bfloat16* kd = qd.k_dst + ((long long)sb * qd.k_seq_rows + pos) * qd.d + (c0 - qd.d);
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c0 + j < rows_b) kd[j] = __float2bfloat16_rn(__uint_as_float(v[j]) + (bias ? bias[c0 + j] : 0.f));
        }
      } else if (r_ok) {
        if (epi == EPI_STORE || epi == EPI_GELU || epi == EPI_QKV) {
          __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out) + (long long)r * ldc + c0;
          if (c0 + 32 <= rows_b && (ldc & 7) == 0) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint32_t pk[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                float x0 = __uint_as_float(v[g * 8 + 2 * e]) + (bias ? bias[c0 + g * 8 + 2 * e] : 0.f);
                float x1 = __uint_as_float(v[g * 8 + 2 * e + 1]) + (bias ? bias[c0 + g * 8 + 2 * e + 1] : 0.f);
                if (epi == EPI_GELU) { x0 = gelu_tanh_fast(x0); x1 = gelu_tanh_fast(x1); }
                __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
                pk[e] = *reinterpret_cast<uint32_t*>(&h2);
              }
              *reinterpret_cast<uint4*>(o + g * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            if (out_lo != nullptr) {   // second half of the hi/lo pair: lo = bf16(x - hi)
              __nv_bfloat16* ol = reinterpret_cast<__nv_bfloat16*>(out_lo) + (long long)r * ldc + c0;
              for (int j = 0; j < 32; ++j) {
                float x = __uint_as_float(v[j]) + (bias ? bias[c0 + j] : 0.f);
                if (epi == EPI_GELU) x = gelu_tanh_fast(x);
                ol[j] = __float2bfloat16_rn(x - __bfloat162float(__float2bfloat16_rn(x)));
              }
            }
          } else {
            for (int j = 0; j < 32; ++j) {
              if (c0 + j < rows_b) {
                float x = __uint_as_float(v[j]) + (bias ? bias[c0 + j] : 0.f);
                if (epi == EPI_GELU) x = gelu_tanh_fast(x);
                const __nv_bfloat16 hi = __float2bfloat16_rn(x);
                o[j] = hi;
                if (out_lo != nullptr)
                  reinterpret_cast<__nv_bfloat16*>(out_lo)[(long long)r * ldc + c0 + j] = __float2bfloat16_rn(x - __bfloat162float(hi));
              }
            }
          }
        } else {
          float* o = reinterpret_cast<float*>(out) + (long long)r * ldc + c0;
          if (epi == EPI_RESIDUAL && !split && c0 + 32 <= rows_b && (ldc & 3) == 0) {
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              float4 h4 = *reinterpret_cast<float4*>(o + g * 4);
              h4.x += __uint_as_float(v[g * 4 + 0]) + (bias ? bias[c0 + g * 4 + 0] : 0.f);
              h4.y += __uint_as_float(v[g * 4 + 1]) + (bias ? bias[c0 + g * 4 + 1] : 0.f);
              h4.z += __uint_as_float(v[g * 4 + 2]) + (bias ? bias[c0 + g * 4 + 2] : 0.f);
              h4.w += __uint_as_float(v[g * 4 + 3]) + (bias ? bias[c0 + g * 4 + 3] : 0.f);
              *reinterpret_cast<float4*>(o + g * 4) = h4;
            }
          } else {
            for (int j = 0; j < 32; ++j) {
              if (c0 + j < rows_b) {
                const float x = __uint_as_float(v[j]) + (bias ? bias[c0 + j] : 0.f);
                if (epi == EPI_RESIDUAL) { if (split) atomicAdd(o + j, x); else o[j] += x; }
                else o[j] = x;
              }
            }
          }
        }
      }
    } else {
      // out[c][r]: c = token, r = feature; consecutive lanes write consecutive features
      // ROLL: a rolled loop over the valid tokens only.  Unrolled 32 times, this body (every epilogue kind, the
      // cache arithmetic of the fused QKV) is tens of kilobytes of straight-line code; a CTA of the one-tile kernel
      // runs through it once, and the few-CTA weight-streaming launches then spend their time fetching instructions
      // (100 KB -> 14 KB of code per kernel).  v[] is then indexed dynamically, i.e. it passes through local memory
      // (32 words per thread).  The persistent kernel repeats its epilogue tile after tile and keeps the unrolled form.
      const float bv = (bias != nullptr && r_ok) ? bias[r] : 0.f;
      auto put = [&](int c, float acc) {
        float x = acc + bv;
        const long long o = (long long)c * ldc + r;
        if (epi == EPI_QKV) {
          if (r < qd.d || (r < 2 * qd.d && qd.k_dst == nullptr)) {
            reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(x);
          } else {
            const int sb = c / qd.rows_per_seq, si = c - sb * qd.rows_per_seq;
            const int cl = qd.ctx_len[sb];
            const int pos = qd.mode == 1 ? cl - 1 + si : si;
            if (qd.mode != 2 || si < cl - 1) {
              if (r < 2 * qd.d) {
                if (pos < qd.k_seq_rows)
                  qd.k_dst[((long long)sb * qd.k_seq_rows + pos) * qd.d + (r - qd.d)] = __float2bfloat16_rn(x);
              } else if (pos < qd.vt_ld) {
                qd.vt_dst[((long long)sb * qd.d + (r - 2 * qd.d)) * qd.vt_ld + pos] = __float2bfloat16_rn(x);
              }
            }
          }
        } else if (epi == EPI_STORE || epi == EPI_GELU) {
          if (epi == EPI_GELU) x = gelu_tanh_fast(x);
          const __nv_bfloat16 hi = __float2bfloat16_rn(x);
          reinterpret_cast<__nv_bfloat16*>(out)[o] = hi;
          if (out_lo != nullptr) reinterpret_cast<__nv_bfloat16*>(out_lo)[o] = __float2bfloat16_rn(x - __bfloat162float(hi));
        }
        else if (epi == EPI_RESIDUAL) { if (split) atomicAdd(reinterpret_cast<float*>(out) + o, x); else reinterpret_cast<float*>(out)[o] += x; }
        else reinterpret_cast<float*>(out)[o] = x;
      };
      if (ROLL) {
        const int jn = rows_b - c0 < 32 ? rows_b - c0 : 32;
        if (r_ok) {
#pragma unroll 1
          for (int j = 0; j < jn; ++j) put(c0 + j, __uint_as_float(v[j]));
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (r_ok && c0 + j < rows_b) put(c0 + j, __uint_as_float(v[j]));
      }
    }
  }
}

// SWAP orientation, fp32 residual stream (tile = 128 features x up to BN tokens; a thread owns one feature): the tile
// is written token-major into four 128-byte-swizzled boxes of 32 features, one per epilogue warp, and leaves as four
// TMA add-reduces, out[token][feature] += acc + bias; tokens past the last row and features past the last column are
// clipped by the tensor map.  (Per-element atomics from the registers -- 4224 a CTA, half a million a launch on 53 k
// addresses under K splits -- took 3.5 us per launch.)
template <int BN>
__device__ __forceinline__ void epilogue_swap_reduce(uint32_t tmem_acc, int m0, int n0, int q, int lane, int rows_a,
                                                     const float* __restrict__ bias, const CUtensorMap* map_out,
                                                     uint8_t* stage_generic, uint32_t stage_u32) {
  const int r = m0 + q * 32 + lane;
  const float bv = (bias != nullptr && r < rows_a) ? bias[r] : 0.f;
  uint8_t* box = stage_generic + q * (BN * 128);
  const uint32_t chunk = (uint32_t)lane >> 2, within = ((uint32_t)lane & 3u) * 4u;
#pragma unroll 1
  for (int cc = 0; cc < BN / 32; ++cc) {
    uint32_t v[32];
    tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 32), v);
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const uint32_t t = (uint32_t)(cc * 32 + j);
      *reinterpret_cast<float*>(box + t * 128u + ((chunk ^ (t & 7u)) << 4) + within) = __uint_as_float(v[j]) + bv;
    }
  }
  fence_async_smem();
  named_bar_sync(2, 128);
  if (threadIdx.x == 64) {
    for (int qq = 0; qq < 4; ++qq)
      if (m0 + qq * 32 < rows_a) tma_reduce_add_2d(map_out, stage_u32 + (uint32_t)(qq * BN * 128), m0 + qq * 32, n0);
    tma_commit_group();
    tma_wait_group_read<0>();       // shared memory stays valid until the copies have read it
  }
}

// ---------------------------------------------------------------------------------------------
// LM-head epilogues that also produce the rows' soft-max statistics (HeadStats): the logits are stored as by
// EPI_STORE_F32, and every (token row, slice of the vocabulary) gets one pair (max z, sum exp(z - max)), z = logit *
// inv_tau -- or (max logit, index of its first occurrence) when inv_tau == 0 -- so that the acceptance step never
// reads the logit matrix for its statistics.
// ---------------------------------------------------------------------------------------------
// Reduction of 32 values per lane across the warp in 31 shuffles: on return a[0] of lane L holds op over all lanes of
// their a[L] (each step halves the values a lane keeps and exchanges the other half with the lane `o` away).
template <typename Op>
__device__ __forceinline__ void warp_reduce_scatter(float (&a)[32], int lane, Op op) {
#pragma unroll
  for (int st = 0; st < 5; ++st) {
    const int o = 16 >> st;            // partner distance = number of values kept
    const bool upper = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if (i < o) {
        const float send = upper ? a[i] : a[i + o];
        const float keep = upper ? a[i + o] : a[i];
        a[i] = op(keep, __shfl_xor_sync(0xffffffffu, send, o));
      }
    }
  }
}
// the same for (value, index) pairs under the arg-max order (ties: lowest index)
__device__ __forceinline__ void warp_reduce_scatter_argmax(float (&a)[32], int (&ix)[32], int lane) {
#pragma unroll
  for (int st = 0; st < 5; ++st) {
    const int o = 16 >> st;
    const bool upper = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      if (i < o) {
        const float send = upper ? a[i] : a[i + o];
        const int send_i = upper ? ix[i] : ix[i + o];
        ArgMax keep;
        keep.s = upper ? a[i + o] : a[i];
        keep.i = upper ? ix[i + o] : ix[i];
        ArgMax got;
        got.s = __shfl_xor_sync(0xffffffffu, send, o);
        got.i = __shfl_xor_sync(0xffffffffu, send_i, o);
        keep = argmax_better(keep, got);
        a[i] = keep.s;
        ix[i] = keep.i;
      }
    }
  }
}

// SWAP orientation (tile = 128 vocabulary rows x up to BN tokens; a thread owns one vocabulary row r): out[token][r]
// = logit.  Each warp reduces its 32 vocabulary rows per token with shuffles; the four warps' pairs meet in shared
// memory (`ex`: [BN / 32][4][32] float2, free between two tiles' epilogues because the four warps pass a common
// barrier before every tile) and warp 0 writes one pair per (token, tile): slice index = tile.
template <int BN>
__device__ __forceinline__ void epilogue_head_swap(uint32_t tmem_acc, int m0, int q, int lane, int V, int tokens,
                                                   float* __restrict__ out, int ldc, const HeadStats& hs, int chunks,
                                                   int tile, float2* ex) {
  const int r = m0 + q * 32 + lane;
  const bool r_ok = r < V;
  const bool greedy = hs.inv_tau == 0.f;
  const float k = hs.inv_tau * 1.4426950408889634f;
  const int n_cc = (tokens + 31) / 32 < BN / 32 ? (tokens + 31) / 32 : BN / 32;
#pragma unroll 1
  for (int cc = 0; cc < n_cc; ++cc) {
    const int c0 = cc * 32;
    uint32_t v[32];
    tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
    float x[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const float acc = __uint_as_float(v[j]);
      if (r_ok && c0 + j < tokens) out[(long long)(c0 + j) * ldc + r] = acc;
      x[j] = r_ok ? acc : -INFINITY;
    }
    float2 pair;
    if (greedy) {
      int ix[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) ix[j] = r_ok ? r : 0x7fffffff;
      warp_reduce_scatter_argmax(x, ix, lane);
      pair = make_float2(x[0], __int_as_float(ix[0]));
    } else {
      float mx[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) mx[j] = x[j];
      warp_reduce_scatter(mx, lane, [](float a, float b) { return fmaxf(a, b); });
      const float m_mine = mx[0];                      // maximum of token c0 + lane over the warp's rows
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float mj = __shfl_sync(0xffffffffu, m_mine, j);
        x[j] = (r_ok && mj > -INFINITY) ? exp2f((x[j] - mj) * k) : 0.f;
      }
      warp_reduce_scatter(x, lane, [](float a, float b) { return a + b; });
      pair = make_float2(m_mine, x[0]);                // (max logit, sum exp((logit - max) * inv_tau))
    }
    ex[(cc * 4 + q) * 32 + lane] = pair;
  }
  named_bar_sync(2, 128);
  if (q == 0) {
    for (int cc = 0; cc < n_cc; ++cc) {
      const int tok = cc * 32 + lane;
      if (tok >= tokens) break;
      float2 a = ex[(cc * 4 + 0) * 32 + lane];
      if (greedy) {
        ArgMax best;
        best.s = a.x; best.i = __float_as_int(a.y);
#pragma unroll
        for (int w = 1; w < 4; ++w) {
          const float2 b = ex[(cc * 4 + w) * 32 + lane];
          ArgMax o;
          o.s = b.x; o.i = __float_as_int(b.y);
          best = argmax_better(best, o);
        }
        a = make_float2(best.s, __int_as_float(best.i));
      } else {
        float m = a.x;
#pragma unroll
        for (int w = 1; w < 4; ++w) m = fmaxf(m, ex[(cc * 4 + w) * 32 + lane].x);
        float sum = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const float2 b = ex[(cc * 4 + w) * 32 + lane];
          if (b.x > -INFINITY) sum += b.y * exp2f((b.x - m) * k);
        }
        a = make_float2(m * hs.inv_tau, sum);
      }
      hs.partial[(long long)tok * chunks + tile] = a;
    }
  }
}

// NORMAL orientation (tile = 128 token rows x BN vocabulary columns; a thread owns one token row): out[r][column] =
// logit, and one pair per (token row, tile): slice index = the tile's index along the vocabulary.
template <int BN>
__device__ __forceinline__ void epilogue_head_normal(uint32_t tmem_acc, int m0, int n0, int q, int lane, int rows, int V,
                                                     float* __restrict__ out, int ldc, const HeadStats& hs, int chunks,
                                                     int n_tile) {
  const int r = m0 + q * 32 + lane;
  const bool r_ok = r < rows;
  const bool greedy = hs.inv_tau == 0.f;
  const float k = hs.inv_tau * 1.4426950408889634f;
  float m = -INFINITY, sum = 0.f;
  int arg = 0x7fffffff;
#pragma unroll 1
  for (int cc = 0; cc < BN / 32; ++cc) {
    const int c0 = n0 + cc * 32;
    if (c0 >= V) break;
    uint32_t v[32];
    tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 32), v);
    float* o = out + (long long)r * ldc + c0;
    float cm = -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const float x = __uint_as_float(v[j]);
      if (c0 + j < V) {
        if (r_ok) o[j] = x;
        if (greedy) { if (x > cm) { cm = x; if (x > m) arg = c0 + j; } }
        else cm = fmaxf(cm, x);
      }
    }
    if (greedy) {
      m = fmaxf(m, cm);
    } else if (cm > -INFINITY) {
      const float m_new = fmaxf(m, cm);
      sum = m == -INFINITY ? 0.f : sum * exp2f((m - m_new) * k);
      m = m_new;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (c0 + j < V) sum += exp2f((__uint_as_float(v[j]) - m) * k);
    }
  }
  if (r_ok) hs.partial[(long long)r * chunks + n_tile] = greedy ? make_float2(m, __int_as_float(arg)) : make_float2(m * hs.inv_tau, sum);
}

// grid = (N tiles, M tiles, K splits).  With more than one K split every CTA accumulates its share of the K
// range and adds it to the fp32 output with atomics (EPI_RESIDUAL only; the bias is added by split 0).
// Tiles of 128 columns or more (NORMAL orientation) are drained by two groups of four epilogue warps, each with half of
// the tile's columns, staging buffers and named barriers of its own: the one-tile kernel cannot overlap its epilogue
// with anything, and a 128 x 256 tile costs four warps several microseconds (one wave of such CTAs is the whole launch).
template <int BN, bool SWAP>
constexpr int one_tile_threads() { return (!SWAP && BN >= 128) ? 320 : THREADS; }

template <int BN, bool SWAP, bool HILO, bool DEEP>
__global__ void __launch_bounds__(one_tile_threads<BN, SWAP>())
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_lo, const __grid_constant__ OutMaps maps_out, int tma_out,
               int rows_a, int rows_b, int K, int epi, const float* __restrict__ bias, void* __restrict__ out,
               void* __restrict__ out_lo, int ldc, int* status, const QkvDst qd, const int* __restrict__ skip) {

  constexpr int STAGES = ring_stages<BN, SWAP, HILO, DEEP>();
  constexpr int STAGE_BYTES = stage_bytes<BN, SWAP, HILO>();
  constexpr int LO_OFF = BM * BK * 2 + BN * BK * 2;     // offset of the lo tile inside a stage
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = base + STAGES * STAGE_BYTES;
  // barrier block: full[STAGES], empty[STAGES], tmem_full, then the TMEM base address and the abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t tmem_full_bar = bar_base + 8u * (2 * STAGES);
  uint8_t* generic_base = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(generic_base + STAGES * STAGE_BYTES + 8 * (2 * STAGES + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(generic_base + STAGES * STAGE_BYTES + 8 * (2 * STAGES + 1) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * BM;      // offset along the A operand's rows (MMA M axis)
  const int n0 = blockIdx.x * BN;      // offset along the B operand's rows (MMA N axis)
  const int total_kb = (K + BK - 1) / BK;
  const int kb_per = (total_kb + (int)gridDim.z - 1) / (int)gridDim.z;
  const int kb0 = (int)blockIdx.z * kb_per;
  const int num_kb = min(kb_per, total_kb - kb0);     // host guarantees >= 1
  const bool split = gridDim.z > 1;
  if (split && blockIdx.z != 0) bias = nullptr;
  constexpr uint32_t TMEM_COLS = BN < 32 ? 32 : BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tmem_full_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TMEM_COLS);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  // Everything above touched only shared / tensor memory; the activations may still be in production.  The weight
  // operand (B, or A in the swapped orientation) is never written while the library runs, so the first fill of the
  // ring with weight tiles starts here, under the tail of the kernel ahead in the stream: the bytes are announced
  // without an arrive, the stage's arrive follows with the activation tiles after the wait.  The early look at the
  // skip flag only decides whether to fetch ahead; a stale value costs time, not correctness.
  constexpr uint32_t W_BYTES = (SWAP ? BM : BN) * BK * 2;
  int n_pre = 0;
  if (threadIdx.x == 0 && (skip == nullptr || *reinterpret_cast<const volatile int*>(skip) == 0)) {
    n_pre = min(num_kb, STAGES);
    for (int kb = 0; kb < n_pre; ++kb) {
      mbar_expect_tx_only(full_bar(kb), W_BYTES);
      const uint32_t sa = base + kb * STAGE_BYTES;
      if (SWAP) tma_load_2d(sa, &map_a, full_bar(kb), (kb0 + kb) * BK, m0);
      else tma_load_2d(sa + BM * BK * 2, &map_b, full_bar(kb), (kb0 + kb) * BK, n0);
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  // The activation tiles of the stages whose weight tiles are already on their way go out at once, before the skip
  // flag has even been read (one L2 round trip that would otherwise sit in front of the first operand tile of every
  // launch of a drafter evaluation); if the evaluation turns out to be skipped the tiles are waited for and dropped.
  if (threadIdx.x == 0) {
    for (int kb = 0; kb < n_pre; ++kb) {
      const uint32_t sa = base + kb * STAGE_BYTES;
      mbar_expect_tx(full_bar(kb), (uint32_t)STAGE_BYTES - W_BYTES);
      if (SWAP) tma_load_2d(sa + BM * BK * 2, &map_b, full_bar(kb), (kb0 + kb) * BK, n0);
      else tma_load_2d(sa, &map_a, full_bar(kb), (kb0 + kb) * BK, m0);
      if (HILO) tma_load_2d(sa + LO_OFF, &map_lo, full_bar(kb), (kb0 + kb) * BK, SWAP ? n0 : m0);
    }
  }
  // launches of a drafter evaluation do nothing when the evaluation is skipped (they still free their TMEM below)
  const bool active = skip == nullptr || *skip == 0;

  if (!active) {
    // tiles fetched ahead must have landed before the CTA gives its shared memory back
    for (int kb = 0; kb < n_pre; ++kb) {
      const long long t0 = clock64();
      while (!mbar_try(full_bar(kb), 0u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
    }
  } else if (warp == 0) {
    if (lane == 0) {
      int issued = n_pre;
      for (int kb = n_pre; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
        const uint32_t sa = base + s * STAGE_BYTES;
        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, status)) break;
        mbar_expect_tx(full_bar(s), (uint32_t)STAGE_BYTES);
        tma_load_2d(sa, &map_a, full_bar(s), (kb0 + kb) * BK, m0);
        tma_load_2d(sa + BM * BK * 2, &map_b, full_bar(s), (kb0 + kb) * BK, n0);
        if (HILO) tma_load_2d(sa + LO_OFF, &map_lo, full_bar(s), (kb0 + kb) * BK, SWAP ? n0 : m0);
        issued = kb + 1;
      }
      if (*abort_flag) {
        // do not leave while copies into this CTA's shared memory may still be in flight
        const int first = issued > STAGES ? issued - STAGES : 0;
        for (int kb = first; kb < issued; ++kb) {
          const long long t0 = clock64();
          while (!mbar_try(full_bar(kb % STAGES), (uint32_t)(kb / STAGES) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc<BN>();
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
        ok = mbar_wait(full_bar(s), ph, abort_flag, status);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = base + s * STAGE_BYTES;
        const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + BM * BK * 2);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k)
          umma(tmem_base, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
               (kb > 0 || k > 0) ? 1u : 0u);
        if (HILO) {
          const uint64_t dl = make_smem_desc(sa + LO_OFF);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            const uint64_t o = (uint64_t)(k * UMMA_K * 2 / 16);
            if (SWAP) umma(tmem_base, da + o, dl + o, idesc, 1u);
            else umma(tmem_base, dl + o, db + o, idesc, 1u);
          }
        }
        umma_commit(empty_bar(s));     // frees the stage once these MMAs have read it
      }
      if (ok) umma_commit(tmem_full_bar);
    }
  } else {
    // epilogue warps own TMEM lane quarters (warp id % 4); with two groups, group g = (warp - 2) / 4 takes the chunks
    // [g * BN / 64, (g + 1) * BN / 64) and the staging buffers at 32 KB * g of the (now idle) operand ring
    const int q = warp & 3;
    constexpr bool TWO = one_tile_threads<BN, SWAP>() == 320;
    const int grp = TWO ? (warp - 2) >> 2 : 0;
    const EpiGroup eg = TWO ? EpiGroup{grp * (BN / 64), (grp + 1) * (BN / 64), 2, 2 + grp, 64 + grp * 128} : whole_tile_group<BN>();
    uint8_t* stage_g = generic_base + grp * (2 * 128 * 128);
    const uint32_t stage_u = base + grp * (2 * 128 * 128);
    // every lane waits; the outcome is made warp-uniform because tcgen05.ld is a warp-wide instruction
    // (and uniform over the four warps of a group, which meet at named barriers in the TMA-store path)
    float* bias_s = reinterpret_cast<float*>(generic_base + STAGES * STAGE_BYTES + 256);
    // tma_out == 2 (fused QKV): only tiles that lie wholly in the columns kept in place (Q, and K without a cache)
    // are plain row-major stores; the others scatter into the K cache / V^T and take the manual path
    // tma_out == 3: also the tiles that lie wholly in V leave by TMA, transposed (drafter; 128-row tiles never
    // straddle sequences there)
    const bool use_tma = !SWAP && (tma_out == 1 || (tma_out >= 2 && n0 + BN <= (qd.k_dst != nullptr ? qd.d : 2 * qd.d)));
    const bool vt_tma = !SWAP && tma_out == 3 && n0 >= 2 * qd.d && n0 + BN <= rows_b;
    if (use_tma || vt_tma) stage_bias(bias_s, bias, n0, rows_b, eg);     // while the main loop runs
    const bool ready = named_bar_and(TWO ? 4 + grp : 1, 128, mbar_wait(tmem_full_bar, 0u, abort_flag, status));
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ready && use_tma) {
      int n_store = 0;
      epilogue_tma<BN>(tmem_base, m0, n0, q, lane, epi == EPI_QKV ? (int)EPI_STORE : epi, bias_s, &maps_out.out, stage_g, stage_u,
                       n_store, eg);
      if ((int)threadIdx.x == eg.first_tid) tma_wait_group_read<0>();      // shared memory stays valid until the copies have read it
    } else if (ready && vt_tma) {
      int n_store = 0;
      const int sb = m0 / qd.rows_per_seq;
      epilogue_vt<BN>(tmem_base, q, lane, bias_s, &maps_out.vt, stage_g, stage_u, n_store, sb * qd.d + (n0 - 2 * qd.d),
                      m0 - sb * qd.rows_per_seq, eg);
      if ((int)threadIdx.x == eg.first_tid) tma_wait_group_read<0>();
    } else if (ready && SWAP && tma_out == 4) {
      if constexpr (SWAP) epilogue_swap_reduce<BN>(tmem_base, m0, n0, q, lane, rows_a, bias, &maps_out.out, generic_base, base);
    } else if (ready) {
      epilogue_manual<BN, SWAP, SWAP>(tmem_base, m0, n0, q, lane, rows_a, rows_b, epi, bias, out, out_lo, ldc, split, qd, eg.c_begin,
                                      eg.c_end);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------
// Persistent variant for grids of many tiles (NORMAL orientation): one CTA per SM walks over tiles
// (tile = blockIdx.x, + gridDim.x, ...; the N index runs fastest when W fits well into L2, so that the CTAs running
// at one time share few A tiles and every A tile comes from DRAM once; else the M index runs fastest).  Two
// accumulators live in TMEM, so the MMA warp fills one while the epilogue warps drain the other; the operand ring
// runs on across tile boundaries.  Extra barriers: tmem_full[2] (MMA -> epilogue), tmem_empty[2] (epilogue -> MMA).
// ---------------------------------------------------------------------------------------------
// SWAP (the LM heads: a few tokens against 50257 weight rows): the tiles are 128 weight rows each and the kernel is a
// weight stream; what the persistent form buys there is that the loads run on while a tile's epilogue stores.
template <int BN, bool HILO, bool SWAP = false>
constexpr int persist_stages() {
  constexpr int s = (227 * 1024 - 2 * 128 * 128 - 1024 - 1024 - 512 - 2048) / stage_bytes<BN, SWAP, HILO>();
  return s > 8 ? 8 : s;
}
template <int BN, bool HILO, bool SWAP = false>
constexpr int persist_smem_bytes() {
  return persist_stages<BN, HILO, SWAP>() * stage_bytes<BN, SWAP, HILO>() + 2 * 128 * 128 + 1024 + 512 + 2048;
}

// STATS: the LM-head instantiations whose epilogue also writes the rows' soft-max statistics (HeadStats); kept apart so
// that the other launches do not carry that code
template <int BN, bool HILO, bool SWAP = false, bool STATS = false>
__global__ void __launch_bounds__(THREADS)
gemm_tc_persist_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                       const __grid_constant__ CUtensorMap map_lo, const __grid_constant__ OutMaps maps_out, int tma_out,
                       int rows_a, int rows_b, int K, int epi, const float* __restrict__ bias, void* __restrict__ out,
                       void* __restrict__ out_lo, int ldc, int* status, const QkvDst qd, const int* __restrict__ skip,
                       int tiles_m, int tiles_n, int n_fastest, const HeadStats hs, int hs_chunks) {
  constexpr int STAGES = persist_stages<BN, HILO, SWAP>();
  constexpr int STAGE_BYTES = stage_bytes<BN, SWAP, HILO>();
  constexpr int LO_OFF = BM * BK * 2 + BN * BK * 2;
  constexpr int STAGING_OFF = STAGES * STAGE_BYTES;
  constexpr int BAR_OFF = STAGING_OFF + 2 * 128 * 128;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* generic_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_base = base + BAR_OFF;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(generic_base + BAR_OFF + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(generic_base + BAR_OFF + 8 * (2 * STAGES + 4) + 8);
  constexpr uint32_t TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (K + BK - 1) / BK;
  const int n_tiles = tiles_m * tiles_n;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 128); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // the first ring fill of weight tiles starts before the wait for the kernel ahead (see gemm_tc_kernel)
  constexpr uint32_t W_BYTES = (SWAP ? BM : BN) * BK * 2;
  int n_pre = 0;
  if (threadIdx.x == 0 && (int)blockIdx.x < n_tiles && (skip == nullptr || *reinterpret_cast<const volatile int*>(skip) == 0)) {
    const long long mine = (long long)((n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x) * num_kb;
    n_pre = (int)(mine < STAGES ? mine : STAGES);
    for (int j = 0; j < n_pre; ++j) {
      const int tile = (int)blockIdx.x + (j / num_kb) * (int)gridDim.x, kb = j % num_kb;
      const int m0 = (n_fastest ? tile / tiles_n : tile % tiles_m) * BM;
      const int n0 = (n_fastest ? tile % tiles_n : tile / tiles_m) * BN;
      mbar_expect_tx_only(full_bar(j), W_BYTES);
      const uint32_t sa = base + j * STAGE_BYTES;
      if (SWAP) tma_load_2d(sa, &map_a, full_bar(j), kb * BK, m0);
      else tma_load_2d(sa + BM * BK * 2, &map_b, full_bar(j), kb * BK, n0);
    }
  }
  pdl_launch_dependents();
  pdl_wait();
  const bool active = skip == nullptr || *skip == 0;

  if (!active) {
    // weight tiles fetched ahead must have landed before the CTA gives its shared memory back
    for (int j = 0; j < n_pre; ++j) {
      mbar_arrive(full_bar(j));
      const long long t0 = clock64();
      while (!mbar_try(full_bar(j), 0u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
    }
  } else if (warp == 0) {
    if (lane == 0) {
      long long it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int m0 = (n_fastest ? tile / tiles_n : tile % tiles_m) * BM;
        const int n0 = (n_fastest ? tile % tiles_n : tile / tiles_m) * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = (int)(it % STAGES);
          const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
          const uint32_t sa = base + s * STAGE_BYTES;
          if (it < n_pre) {
            mbar_expect_tx(full_bar(s), (uint32_t)STAGE_BYTES - W_BYTES);    // the weight tile is already on its way
            if (SWAP) tma_load_2d(sa + BM * BK * 2, &map_b, full_bar(s), kb * BK, n0);
            else tma_load_2d(sa, &map_a, full_bar(s), kb * BK, m0);
          } else {
            if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, status)) { ok = false; break; }
            mbar_expect_tx(full_bar(s), (uint32_t)STAGE_BYTES);
            tma_load_2d(sa, &map_a, full_bar(s), kb * BK, m0);
            tma_load_2d(sa + BM * BK * 2, &map_b, full_bar(s), kb * BK, n0);
          }
          if (HILO) tma_load_2d(sa + LO_OFF, &map_lo, full_bar(s), kb * BK, SWAP ? n0 : m0);   // the activation side
        }
      }
      if (*abort_flag) {
        // do not leave while copies into this CTA's shared memory may still be in flight
        for (long long j = it > STAGES ? it - STAGES : 0; j < it; ++j) {
          const long long t0 = clock64();
          while (!mbar_try(full_bar((int)(j % STAGES)), (uint32_t)(j / STAGES) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc<BN>();
      long long it = 0;
      int i = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++i) {
        const int buf = i & 1;
        ok = mbar_wait(tempty_bar(buf), ((uint32_t)(i >> 1) & 1u) ^ 1u, abort_flag, status);   // accumulator drained
        if (!ok) break;
        fence_after_sync();
        const uint32_t acc = tmem_base + (uint32_t)(buf * BN);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = (int)(it % STAGES);
          ok = mbar_wait(full_bar(s), (uint32_t)(it / STAGES) & 1u, abort_flag, status);
          if (!ok) break;
          fence_after_sync();
          const uint32_t sa = base + s * STAGE_BYTES;
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + BM * BK * 2);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma(acc, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          if (HILO) {
            const uint64_t dl = make_smem_desc(sa + LO_OFF);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              const uint64_t o = (uint64_t)(k * UMMA_K * 2 / 16);
              if (SWAP) umma(acc, da + o, dl + o, idesc, 1u);
              else umma(acc, dl + o, db + o, idesc, 1u);
            }
          }
          umma_commit(empty_bar(s));
        }
        if (ok) umma_commit(tfull_bar(buf));
      }
    }
  } else {
    const int q = warp & 3;
    int n_store = 0, i = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++i) {
      const int buf = i & 1;
      const int m0 = (n_fastest ? tile / tiles_n : tile % tiles_m) * BM;
      const int n0 = (n_fastest ? tile % tiles_n : tile / tiles_m) * BN;
      float* bias_s = reinterpret_cast<float*>(generic_base + BAR_OFF + 512) + buf * BN;
      const bool use_tma = !SWAP && (tma_out == 1 || (tma_out >= 2 && n0 + BN <= (qd.k_dst != nullptr ? qd.d : 2 * qd.d)));
      const bool vt_tma = !SWAP && tma_out == 3 && n0 >= 2 * qd.d && n0 + BN <= rows_b;
      if (use_tma || vt_tma) stage_bias<BN>(bias_s, bias, n0, rows_b);  // while the tile's main loop runs
      const bool ready = named_bar_and(1, 128, mbar_wait(tfull_bar(buf), (uint32_t)(i >> 1) & 1u, abort_flag, status));
      if (!ready) break;
      fence_after_sync();
      const uint32_t acc = tmem_base + (uint32_t)(buf * BN);
      if constexpr (STATS && SWAP)       // LM head: logits + their soft-max statistics (the staging buffers are free here)
        epilogue_head_swap<BN>(acc, m0, q, lane, rows_a, rows_b, reinterpret_cast<float*>(out), ldc, hs, hs_chunks, m0 / BM,
                               reinterpret_cast<float2*>(generic_base + STAGING_OFF));
      else if constexpr (STATS)
        epilogue_head_normal<BN>(acc, m0, n0, q, lane, rows_a, rows_b, reinterpret_cast<float*>(out), ldc, hs, hs_chunks, n0 / BN);
      else if (SWAP)
        epilogue_manual<BN, true>(acc, m0, n0, q, lane, rows_a, rows_b, epi, bias, out, out_lo, ldc, false, qd);
      else if (use_tma)
        epilogue_tma<BN>(acc, m0, n0, q, lane, epi == EPI_QKV ? (int)EPI_STORE : epi, bias_s, &maps_out.out,
                         generic_base + STAGING_OFF, base + STAGING_OFF, n_store);
      else if (vt_tma)
        epilogue_vt<BN>(acc, q, lane, bias_s, &maps_out.vt, generic_base + STAGING_OFF, base + STAGING_OFF, n_store,
                        (m0 / qd.rows_per_seq) * qd.d + (n0 - 2 * qd.d), m0 % qd.rows_per_seq);
      else
        epilogue_manual<BN, false>(acc, m0, n0, q, lane, rows_a, rows_b, epi, bias, out, out_lo, ldc, false, qd);
      // this thread's reads of the accumulator are complete (tcgen05.wait::ld inside tmem_ld32): hand it back
      fence_before_sync();
      mbar_arrive(tempty_bar(buf));
    }
    if (threadIdx.x == 64) tma_wait_group_read<0>();      // staging memory stays valid until the copies have read it
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    fence_after_sync();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------
// CTA-pair variant of the persistent kernel (tcgen05 cta_group::2): a cluster of two CTAs on two SMs owns a 256 x 256
// tile.  CTA r loads rows m0 + 128 r of A and rows n0 + 128 r of W (half of the B tile) into its own shared memory;
// one thread of CTA 0 (the leader) issues MMAs that run on both SMs' tensor cores, each reading its own A half and
// both B halves, and accumulating the CTA's 128 x 256 half of the result in its own TMEM.  Per 64-wide k-block a CTA
// fills 32 KB instead of the 48 KB of a one-CTA 128 x 256 tile, which lifts the shared-memory-fill bound from 2/3 of
// the tensor peak to the peak.  Every barrier is an mbarrier in one CTA's shared memory; what the other CTA has to
// learn is forwarded by a thread with a remote arrive:
//   full[s]   (leader only: 1 arrive + the bytes of both CTAs' copies) -- both producers name the leader's barrier in
//             their TMA loads (cta_group::2 form); the leader's producer announces the bytes of both
//   empty[s]  (both: 1 arrive) -- the leader's MMA thread commits once to its own barrier and once to the peer's
//   tfull[b]  (both: 1 arrive) -- leader's commit locally; its epilogue thread 64 forwards it to the peer
//   tempty[b] (leader: 16 arrives) -- the epilogue warps of both CTAs arrive on the leader's barrier
// (with forwarding threads on the full / empty path the refill round trip exceeded what the ring covers and the
// kernel ran at half speed)
// The epilogues are those of the one-CTA kernels, applied by each CTA to its half; eight epilogue warps in two groups
// (columns 0..127 and 128..255, one staging buffer each), because the main loop of a tile is a third shorter here.  The CTAs meet at a cluster
// barrier before TMEM is freed, so that neither leaves while the other may still touch its shared memory.
// ---------------------------------------------------------------------------------------------
constexpr int PAIR_STAGE_BYTES = BM * BK * 2 + 128 * BK * 2;     // A tile + half of the 256-wide B tile: 32 KB
constexpr int PAIR_STAGES = 6;
constexpr int PAIR_STAGING_OFF = PAIR_STAGES * PAIR_STAGE_BYTES;
constexpr int PAIR_BAR_OFF = PAIR_STAGING_OFF + 2 * 128 * 128;
constexpr int PAIR_SMEM = PAIR_BAR_OFF + 512 + 1024 + 1024;       // barriers, one tile's bias, alignment slack

constexpr int PAIR_THREADS = 320;   // warp 0: TMA, warp 1: MMA (leader) + TMEM owner, warps 2-5 and 6-9: two epilogue groups

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PAIR_THREADS)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ OutMaps maps_out, int tma_out, int rows_a, int rows_b, int K, int epi,
                    const float* __restrict__ bias, void* __restrict__ out, int ldc, int* status, const QkvDst qd,
                    const int* __restrict__ skip, int tiles_m2, int tiles_n, int n_fastest) {
  constexpr int BN = 256;
  constexpr int STAGES = PAIR_STAGES;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* generic_base = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bar_base = base + PAIR_BAR_OFF;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(generic_base + PAIR_BAR_OFF + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(generic_base + PAIR_BAR_OFF + 8 * (2 * STAGES + 4) + 8);
  constexpr uint32_t TMEM_COLS = 512;                // two 256-column accumulators

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const uint32_t peer = rank ^ 1u;
  const int num_kb = (K + BK - 1) / BK;
  const int n_tiles = tiles_m2 * tiles_n;
  const int pair = (int)(blockIdx.x >> 1), n_pairs = (int)(gridDim.x >> 1);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 16); }   // one arrive per epilogue warp of the pair
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  cluster_sync_all();                                // both CTAs' barriers exist before anyone arrives remotely
  if (warp == 1) tmem_alloc_pair(tmem_slot, TMEM_COLS);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_launch_dependents();
  pdl_wait();
  const bool active = skip == nullptr || *skip == 0;   // the same value in both CTAs (read after the producer grid)

  if (!active) {
  } else if (warp == 0) {
    if (lane == 0) {
      long long it = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs) {
        const int m0 = (n_fastest ? tile / tiles_n : tile % tiles_m2) * (2 * BM) + (int)rank * BM;
        const int n0 = (n_fastest ? tile % tiles_n : tile / tiles_m2) * BN + (int)rank * 128;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = (int)(it % STAGES);
          const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
          if (!mbar_wait_cluster(empty_bar(s), ph ^ 1u, abort_flag, status)) { ok = false; break; }
          if (leader) mbar_expect_tx(full_bar(s), 2u * (uint32_t)PAIR_STAGE_BYTES);   // both CTAs' bytes
          const uint32_t lf = map_to_cta(full_bar(s), 0u);
          const uint32_t sa = base + s * PAIR_STAGE_BYTES;
          tma_load_2d_pair(sa, &map_a, lf, kb * BK, m0);
          tma_load_2d_pair(sa + BM * BK * 2, &map_b, lf, kb * BK, n0);
        }
      }
      if (leader && *abort_flag) {
        // do not leave while copies into the pair's shared memory may still be in flight (the peer stays until the
        // cluster barrier at the end, which the leader reaches after this)
        for (long long j = it > STAGES ? it - STAGES : 0; j < it; ++j) {
          const long long t0 = clock64();
          while (!mbar_try_cluster(full_bar((int)(j % STAGES)), (uint32_t)(j / STAGES) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
      long long it = 0;
      int i = 0;
      bool ok = true;
      for (int tile = pair; tile < n_tiles && ok; tile += n_pairs, ++i) {
        const int buf = i & 1;
        ok = mbar_wait_cluster(tempty_bar(buf), ((uint32_t)(i >> 1) & 1u) ^ 1u, abort_flag, status);   // drained in both CTAs
        if (!ok) break;
        fence_after_sync();
        const uint32_t acc = tmem_base + (uint32_t)(buf * BN);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = (int)(it % STAGES);
          ok = mbar_wait_cluster(full_bar(s), (uint32_t)(it / STAGES) & 1u, abort_flag, status);
          if (!ok) break;
          fence_after_sync();
          const uint32_t sa = base + s * PAIR_STAGE_BYTES;
          const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + BM * BK * 2);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_pair(acc, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit_pair(empty_bar(s));                       // frees the stage in this CTA ...
          umma_commit_pair(map_to_cta(empty_bar(s), peer));     // ... and in the peer
        }
        if (ok) umma_commit_pair(tfull_bar(buf));
      }
    }
  } else {
    // two groups of four warps; each drains half of the tile's columns through a staging buffer of its own
    const int q = warp & 3;
    const int grp = (warp - 2) >> 2;
    const EpiGroup eg{grp * 4, grp * 4 + 4, 1, 2 + grp, 64 + grp * 128};
    uint8_t* stage_g = generic_base + PAIR_STAGING_OFF + grp * (128 * 128);
    const uint32_t stage_u = base + PAIR_STAGING_OFF + grp * (128 * 128);
    int n_store = 0, i = 0;
    const uint32_t leader_tempty0 = map_to_cta(tempty_bar(0), 0u);
    for (int tile = pair; tile < n_tiles; tile += n_pairs, ++i) {
      const int buf = i & 1;
      const int m0 = (n_fastest ? tile / tiles_n : tile % tiles_m2) * (2 * BM) + (int)rank * BM;
      const int n0 = (n_fastest ? tile % tiles_n : tile / tiles_m2) * BN;
      float* bias_s = reinterpret_cast<float*>(generic_base + PAIR_BAR_OFF + 512);   // reused: the same threads read it last
      const bool use_tma = tma_out == 1 || (tma_out >= 2 && n0 + BN <= (qd.k_dst != nullptr ? qd.d : 2 * qd.d));
      const bool vt_tma = tma_out == 3 && n0 >= 2 * qd.d && n0 + BN <= rows_b;
      if (use_tma || vt_tma) stage_bias(bias_s, bias, n0, rows_b, eg);  // while the tile's main loop runs
      const bool mine = mbar_wait_cluster(tfull_bar(buf), (uint32_t)(i >> 1) & 1u, abort_flag, status);
      // the leader forwards "accumulator complete" to the peer's epilogue warps
      if (leader && threadIdx.x == 64 && mine) mbar_arrive_remote_relaxed(map_to_cta(tfull_bar(buf), peer));
      const bool ready = named_bar_and(4 + grp, 128, mine);
      if (!ready) break;
      fence_after_sync();
      const uint32_t acc = tmem_base + (uint32_t)(buf * BN);
      if (use_tma)
        epilogue_tma<BN>(acc, m0, n0, q, lane, epi == EPI_QKV ? (int)EPI_STORE : epi, bias_s, &maps_out.out, stage_g, stage_u,
                         n_store, eg);
      else if (vt_tma)
        epilogue_vt<BN>(acc, q, lane, bias_s, &maps_out.vt, stage_g, stage_u, n_store,
                        (m0 / qd.rows_per_seq) * qd.d + (n0 - 2 * qd.d), m0 % qd.rows_per_seq, eg);
      else
        epilogue_manual<BN, false>(acc, m0, n0, q, lane, rows_a, rows_b, epi, bias, out, nullptr, ldc, false, qd, eg.c_begin,
                                   eg.c_end);
      // the warp's reads of the accumulator are complete (tcgen05.wait::ld inside tmem_ld32): hand it back, one arrive
      // per warp
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_remote_relaxed(leader_tempty0 + 8u * (uint32_t)buf);
    }
    if ((int)threadIdx.x == eg.first_tid) tma_wait_group_read<0>();   // staging memory stays valid until the copies have read it
  }
  fence_before_sync();
  __syncthreads();
  cluster_sync_all();                                // the peer's MMAs, copies and remote arrives are behind us
  if (warp == 1) {
    fence_after_sync();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------------
// The error path of the kernels above, run on purpose: one CTA with their role layout in which nothing ever fills
// the first ring stage.  The MMA role's bounded wait on full[0] runs out after `limit` clocks; it raises the abort
// flag and the status word; the epilogue warps, which wait for the accumulator, see the flag and leave; the producer
// finds the flag, has no copy in flight to wait for, and leaves; TMEM is freed; the CTA returns.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(THREADS) wait_timeout_probe_kernel(long long limit, int* status) {
  __shared__ __align__(8) unsigned long long bars[3];   // full[0], empty[0], tmem_full
  __shared__ uint32_t tmem_slot_s;
  __shared__ int abort_s;
  const uint32_t full0 = smem_u32(&bars[0]), empty0 = smem_u32(&bars[1]), tmem_full = smem_u32(&bars[2]);
  volatile int* abort_flag = &abort_s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(full0, 1); mbar_init(empty0, 1); mbar_init(tmem_full, 1);
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&tmem_slot_s, 32);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = tmem_slot_s;
  pdl_launch_dependents();
  pdl_wait();
  if (warp == 0) {
    // the producer, at the point where it wants to refill a stage: it waits for the MMA that would free it, which
    // never comes; it leaves on the abort flag or on its own limit, with no copy in flight
    if (lane == 0) mbar_wait(empty0, 0u, abort_flag, status, limit);
  } else if (warp == 1) {
    if (lane == 0) {
      const bool ok = mbar_wait(full0, 0u, abort_flag, status, limit);   // nothing arrives: runs out
      if (ok) umma_commit(tmem_full);
    }
  } else {
    const bool ready = named_bar_and(1, 128, mbar_wait(tmem_full, 0u, abort_flag, status, limit));
    (void)ready;                                                         // never true here: no accumulator to drain
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    fence_after_sync();
    tmem_dealloc(tmem_base, 32);
  }
}

// ---------------------------------------------------------------------------------------------
// host side: tensor maps (cached per pointer / shape / box) and launch
// ---------------------------------------------------------------------------------------------
template <int BN, bool SWAP, bool HILO, bool DEEP>
static cudaError_t launch_cfg2(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ml, const OutMaps& mo,
                              int tma_out, int rows_a, int rows_b, int K, int epi, const float* bias, void* out, void* out_lo,
                              int ldc, int* status, cudaStream_t st, const QkvDst& qd, int splits, const int* skip) {
  dim3 grid((rows_b + BN - 1) / BN, (rows_a + BM - 1) / BM, splits);
  launch_k(gemm_tc_kernel<BN, SWAP, HILO, DEEP>, grid, dim3(one_tile_threads<BN, SWAP>()), smem_bytes<BN, SWAP, HILO, DEEP>(), st, ma, mb, ml, mo, tma_out,
           rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status, qd, skip);
  return cudaGetLastError();
}
template <int BN, bool SWAP, bool HILO>
static cudaError_t launch_cfg(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ml, const OutMaps& mo,
                              int tma_out, int rows_a, int rows_b, int K, int epi, const float* bias, void* out, void* out_lo,
                              int ldc, int* status, cudaStream_t st, const QkvDst& qd, int splits, const int* skip) {
  // more than two waves of CTAs: shallow rings, two CTAs per SM (needs 2 x BN TMEM columns <= 512: always true)
  const long long ctas = (long long)((rows_b + BN - 1) / BN) * ((rows_a + BM - 1) / BM) * splits;
  if (ctas > 2 * 148)
    return launch_cfg2<BN, SWAP, HILO, false>(ma, mb, ml, mo, tma_out, rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status,
                                              st, qd, splits, skip);
  return launch_cfg2<BN, SWAP, HILO, true>(ma, mb, ml, mo, tma_out, rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status, st,
                                           qd, splits, skip);
}
template <int BN, bool HILO>
static cudaError_t launch_persist(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ml, const OutMaps& mo,
                                  int tma_out, int rows_a, int rows_b, int K, int epi, const float* bias, void* out,
                                  void* out_lo, int ldc, int* status, cudaStream_t st, const QkvDst& qd, const int* skip,
                                  const HeadStats& hs = HeadStats{}) {
  const int tiles_m = (rows_a + BM - 1) / BM, tiles_n = (rows_b + BN - 1) / BN;
  const long long tiles = (long long)tiles_m * tiles_n;
  const unsigned grid = (unsigned)(tiles < 148 ? tiles : 148);
  const int n_fastest = (long long)rows_b * K * 2 <= (48ll << 20) ? 1 : 0;
  if (hs.partial != nullptr)
    launch_k(gemm_tc_persist_kernel<BN, HILO, false, true>, dim3(grid), dim3(THREADS), persist_smem_bytes<BN, HILO>(), st, ma, mb, ml, mo,
             tma_out, rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status, qd, skip, tiles_m, tiles_n, n_fastest, hs, tiles_n);
  else
    launch_k(gemm_tc_persist_kernel<BN, HILO>, dim3(grid), dim3(THREADS), persist_smem_bytes<BN, HILO>(), st, ma, mb, ml, mo,
             tma_out, rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status, qd, skip, tiles_m, tiles_n, n_fastest, hs, tiles_n);
  return cudaGetLastError();
}

template <int BN, bool HILO>
static cudaError_t launch_persist_swap(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ml, const OutMaps& mo,
                                       int rows_a, int rows_b, int K, int epi, const float* bias, void* out, void* out_lo,
                                       int ldc, int* status, cudaStream_t st, const QkvDst& qd, const int* skip,
                                       const HeadStats& hs) {
  const int tiles_m = (rows_a + BM - 1) / BM, tiles_n = (rows_b + BN - 1) / BN;
  const long long tiles = (long long)tiles_m * tiles_n;
  const unsigned grid = (unsigned)(tiles < 148 ? tiles : 148);
  if (hs.partial != nullptr)
    launch_k(gemm_tc_persist_kernel<BN, HILO, true, true>, dim3(grid), dim3(THREADS), persist_smem_bytes<BN, HILO, true>(), st, ma, mb,
             ml, mo, 0, rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status, qd, skip, tiles_m, tiles_n, 0, hs, tiles_m);
  else
    launch_k(gemm_tc_persist_kernel<BN, HILO, true>, dim3(grid), dim3(THREADS), persist_smem_bytes<BN, HILO, true>(), st, ma, mb, ml,
             mo, 0, rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status, qd, skip, tiles_m, tiles_n, 0, hs, tiles_m);
  return cudaGetLastError();
}

template <int BN, bool SWAP>
static cudaError_t launch_hl(bool hilo, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& ml,
                             const OutMaps& mo, int tma_out, int rows_a, int rows_b, int K, int epi, const float* bias,
                             void* out, void* out_lo, int ldc, int* status, cudaStream_t st, const QkvDst& qd, int splits,
                             const int* skip) {
  if (hilo)
    return launch_cfg<BN, SWAP, true>(ma, mb, ml, mo, tma_out, rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status, st, qd, splits, skip);
  return launch_cfg<BN, SWAP, false>(ma, mb, ml, mo, tma_out, rows_a, rows_b, K, epi, bias, out, out_lo, ldc, status, st, qd, splits, skip);
}

template <int BN, bool SWAP>
static cudaError_t prepare_one() {
  cudaError_t e;
#define SDD_PREP(HILO, DEEP)                                                                                      \
  e = cudaFuncSetAttribute(gemm_tc_kernel<BN, SWAP, HILO, DEEP>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                           smem_bytes<BN, SWAP, HILO, DEEP>());                                                \
  if (e != cudaSuccess) return e;
  SDD_PREP(false, true) SDD_PREP(false, false) SDD_PREP(true, true) SDD_PREP(true, false)
#undef SDD_PREP
  return cudaSuccess;
}

}  // namespace tc

// raise the dynamic shared-memory limit of every kernel variant (once per device, outside any stream capture)
cudaError_t tc_prepare_gemm() {
  using namespace tc;
  cudaError_t e;
  if ((e = prepare_one<32, false>()) != cudaSuccess) return e;
  if ((e = prepare_one<64, false>()) != cudaSuccess) return e;
  if ((e = prepare_one<128, false>()) != cudaSuccess) return e;
  if ((e = prepare_one<256, false>()) != cudaSuccess) return e;
  if ((e = prepare_one<32, true>()) != cudaSuccess) return e;
  if ((e = prepare_one<64, true>()) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_persist_kernel<256, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                persist_smem_bytes<256, false>())) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_persist_kernel<256, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                persist_smem_bytes<256, true>())) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_persist_kernel<256, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                persist_smem_bytes<256, false>())) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(gemm_tc_persist_kernel<256, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                persist_smem_bytes<256, true>())) != cudaSuccess) return e;
#define SDD_PREP_PS(BN_, HL_)                                                                                              \
  if ((e = cudaFuncSetAttribute(gemm_tc_persist_kernel<BN_, HL_, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,        \
                                persist_smem_bytes<BN_, HL_, true>())) != cudaSuccess) return e;                            \
  if ((e = cudaFuncSetAttribute(gemm_tc_persist_kernel<BN_, HL_, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                                persist_smem_bytes<BN_, HL_, true>())) != cudaSuccess) return e;
  SDD_PREP_PS(32, false) SDD_PREP_PS(32, true) SDD_PREP_PS(64, false) SDD_PREP_PS(64, true)
#undef SDD_PREP_PS
  return cudaFuncSetAttribute(gemm_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PAIR_SMEM);
}

static PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
static std::mutex g_map_mu;
static std::map<std::tuple<const void*, long long, long long, long long, int>, CUtensorMap> g_maps;

cudaError_t get_tensor_map(const void* ptr, long long rows, long long cols, long long ld, int box_rows, int box_cols,
                           CUtensorMap* out, int elem_bytes) {
  std::lock_guard<std::mutex> lock(g_map_mu);
  if (g_encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
    g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
  }
  auto key = std::make_tuple(ptr, rows, cols, ld, (box_rows * 1024 + box_cols) * 8 + elem_bytes);
  auto it = g_maps.find(key);
  if (it != g_maps.end()) { *out = it->second; return cudaSuccess; }
  if ((reinterpret_cast<uintptr_t>(ptr) & 15u) != 0 || (ld * elem_bytes) % 16 != 0 || box_cols * elem_bytes > 128 ||
      (elem_bytes != 2 && elem_bytes != 4))
    return cudaErrorInvalidValue;
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * elem_bytes};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(&m, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  if (g_maps.size() > 8192) g_maps.clear();
  g_maps[key] = m;
  *out = m;
  return cudaSuccess;
}

int head_stats_chunks_max(int V) { return (V + tc::BM - 1) / tc::BM; }

cudaError_t launch_wait_timeout_probe(long long limit_cycles, int* status, cudaStream_t st) {
  launch_k(tc::wait_timeout_probe_kernel, dim3(1), dim3(tc::THREADS), 0, st, limit_cycles, status);
  return cudaGetLastError();
}

// A: activations [M rows used, capacity a_cap rows, K], W: weights [N, K]; both dense bf16.
cudaError_t launch_gemm_tc(const __nv_bfloat16* A, long long a_cap, const __nv_bfloat16* W, const float* bias, int M, int N,
                           int K, int epi, void* out, int ldc, int bn_hint, int* status, cudaStream_t st, const QkvDst* qkv,
                           const __nv_bfloat16* A_lo, void* out_lo, const int* skip, const HeadStats* stats, int* stats_chunks) {
  using namespace tc;
  if (stats_chunks != nullptr) *stats_chunks = 0;
  if (M <= 0 || N <= 0) return cudaSuccess;
  // soft-max statistics from the epilogue: fp32 logit stores on a persistent kernel, if the caller's buffer has room
  auto stats_for = [&](int chunks) -> HeadStats {
    HeadStats none = {};
    if (stats == nullptr || stats->partial == nullptr || epi != EPI_STORE_F32 || bias != nullptr || chunks > stats->chunks_capacity)
      return none;
    if (stats_chunks != nullptr) *stats_chunks = chunks;
    return *stats;
  };
  static std::once_flag once;
  static cudaError_t prep = cudaSuccess;
  std::call_once(once, [] { prep = tc_prepare_gemm(); });
  if (prep != cudaSuccess) return prep;
  QkvDst qd = {};
  if (epi == EPI_QKV) {
    if (qkv == nullptr || (qkv->d & 63) != 0) return cudaErrorInvalidValue;
    qd = *qkv;
  }
  CUtensorMap ma, mb, ml;
  cudaError_t e;
  const bool hilo = A_lo != nullptr;
  if (out_lo != nullptr && epi != EPI_STORE && epi != EPI_GELU) return cudaErrorInvalidValue;
  const int total_kb = (K + BK - 1) / BK;
  constexpr int SMS = 148;
  // K splits fill idle SMs of a single-wave grid; only the residual epilogue can add partial sums
  auto pick_splits = [&](long long ctas, int min_kb) {
    if (epi != EPI_RESIDUAL || ctas >= SMS) return 1;
    long long s = SMS / ctas;
    if (s > total_kb / min_kb) s = total_kb / min_kb;
    if (s < 1) s = 1;
    // no empty split: ceil(total_kb / s) * (s - 1) < total_kb
    while (s > 1 && ((total_kb + s - 1) / s) * (s - 1) >= total_kb) --s;
    return (int)s;
  };
  if (M <= 64) {
    // SWAP: A operand = weights (box 128 rows), B operand = tokens (box BN rows)
    const int bn = M <= 32 ? 32 : 64;
    const int splits = pick_splits((N + BM - 1) / BM, 2);
    if ((e = get_tensor_map(W, N, K, K, BM, BK, &ma)) != cudaSuccess) return e;
    if ((e = get_tensor_map(A, a_cap, K, K, bn, BK, &mb)) != cudaSuccess) return e;
    ml = mb;
    if (hilo && (e = get_tensor_map(A_lo, a_cap, K, K, bn, BK, &ml)) != cudaSuccess) return e;
    OutMaps none;
    none.out = ma; none.vt = ma;
    // fp32 residual stream with 16-byte-aligned rows: the tile leaves as TMA add-reduces (see epilogue_swap_reduce)
    int swap_tma = 0;
    if (epi == EPI_RESIDUAL && (ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(out) & 15u) == 0) {
      if ((e = get_tensor_map(out, M, N, ldc, bn, 32, &none.out, 4)) != cudaSuccess) return e;
      swap_tma = 4;
    }
    // many weight tiles (the LM heads): the persistent kernel keeps the weight stream going across tiles
    // (SDD_GEMM_PERSIST=0 switches it off)
    {
      const char* pe = getenv("SDD_GEMM_PERSIST");
      if ((pe == nullptr || atoi(pe) != 0) && splits == 1 && (N + BM - 1) / BM > 2 * SMS) {
        const HeadStats hs = stats_for((N + BM - 1) / BM);
        if (bn == 32)
          return hilo ? launch_persist_swap<32, true>(ma, mb, ml, none, N, M, K, epi, bias, out, out_lo, ldc, status, st, qd, skip, hs)
                      : launch_persist_swap<32, false>(ma, mb, ml, none, N, M, K, epi, bias, out, out_lo, ldc, status, st, qd, skip, hs);
        return hilo ? launch_persist_swap<64, true>(ma, mb, ml, none, N, M, K, epi, bias, out, out_lo, ldc, status, st, qd, skip, hs)
                    : launch_persist_swap<64, false>(ma, mb, ml, none, N, M, K, epi, bias, out, out_lo, ldc, status, st, qd, skip, hs);
      }
    }
    if (bn == 32) return launch_hl<32, true>(hilo, ma, mb, ml, none, swap_tma, N, M, K, epi, bias, out, out_lo, ldc, status, st, qd, splits, skip);
    return launch_hl<64, true>(hilo, ma, mb, ml, none, swap_tma, N, M, K, epi, bias, out, out_lo, ldc, status, st, qd, splits, skip);
  }
  int bn = bn_hint == 512 ? 256 : bn_hint;       // 512: the CTA-pair kernel on 256 x 256 tiles
  const long long mt = (M + BM - 1) / BM;
  int splits = 1;
  if (bn != 32 && bn != 64 && bn != 128 && bn != 256) {
    // Tile width (and K splits) by a cost model in SM clocks.  A CTA's main loop is bound by the fill rate of its
    // shared memory (about 64 bytes per clock): (128 + bn) * 128 bytes per 64-wide k-block, i.e. 2 * (128 + bn) clocks,
    // against 2 * bn clocks of tensor-core time.  CTAs that share an SM share that rate, so a grid costs
    // ceil(CTAs / SMs) times one CTA; the epilogue adds a term that grows with the tile width.  Wide tiles with more
    // K splits therefore beat narrow tiles whenever the grid would otherwise leave SMs idle.
    double best = 0.0;
    for (int cand : {256, 128, 64, 32}) {
      const long long ctas1 = mt * ((N + cand - 1) / cand);
      const int s = pick_splits(ctas1, 4);
      const int kb_per = (total_kb + s - 1) / s;
      const long long waves = (ctas1 * s + SMS - 1) / SMS;
      double cost = (double)waves * (2.0 * (128 + cand) * kb_per + 600.0 + 8.0 * cand);
      if (cand == 32 && epi != EPI_RESIDUAL && epi != EPI_STORE_F32) cost += (double)waves * 3000.0;   // no TMA store at this width
      if (best == 0.0 || cost < best * 0.97) { best = cost; bn = cand; splits = s; }
    }
  } else {
    splits = pick_splits(mt * ((N + bn - 1) / bn), 4);
  }
  if ((e = get_tensor_map(A, a_cap, K, K, BM, BK, &ma)) != cudaSuccess) return e;
  if ((e = get_tensor_map(W, N, K, K, bn, BK, &mb)) != cudaSuccess) return e;
  ml = ma;
  if (hilo && (e = get_tensor_map(A_lo, a_cap, K, K, BM, BK, &ml)) != cudaSuccess) return e;
  // output through TMA where the layout allows 16-byte-aligned rows (see the kernel's epilogue)
  OutMaps mo;
  mo.out = ma; mo.vt = ma;
  int tma_out = 0;
  if (epi == EPI_RESIDUAL && (ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(out) & 15u) == 0) {
    if ((e = get_tensor_map(out, M, N, ldc, BM, 32, &mo.out, 4)) != cudaSuccess) return e;
    tma_out = 1;
  } else if ((epi == EPI_STORE || epi == EPI_GELU || epi == EPI_QKV) && out_lo == nullptr && bn >= 64 && (ldc & 7) == 0 &&
             (reinterpret_cast<uintptr_t>(out) & 15u) == 0) {
    if ((e = get_tensor_map(out, M, N, ldc, BM, 64, &mo.out, 2)) != cudaSuccess) return e;
    tma_out = epi == EPI_QKV ? 2 : 1;   // fused QKV: per tile, see the kernel
    // drafter (every row of a tile is a position of one sequence, all of them stored): V tiles by TMA too
    if (epi == EPI_QKV && qd.mode == 0 && qd.vt_dst != nullptr && (M % BM) == 0 && (qd.rows_per_seq % BM) == 0 &&
        (qd.vt_ld & 7) == 0 && (reinterpret_cast<uintptr_t>(qd.vt_dst) & 15u) == 0 && qd.rows_per_seq <= qd.vt_ld) {
      if ((e = get_tensor_map(qd.vt_dst, (long long)(M / qd.rows_per_seq) * qd.d, qd.vt_ld, qd.vt_ld, 64, 64, &mo.vt, 2)) !=
          cudaSuccess)
        return e;
      tma_out = 3;
    }
  }
  // CTA pairs on 256 x 256 tiles for the large GEMMs (bn_hint 512 forces them, SDD_GEMM_PAIR=0 switches them off, =2 drops the size rule)
  {
    const char* pe = getenv("SDD_GEMM_PAIR");
    const bool pair_on = pe == nullptr || atoi(pe) != 0;
    const bool pair_any_size = pe != nullptr && atoi(pe) == 2;      // tests: pairs wherever they are eligible
    const bool eligible = !hilo && out_lo == nullptr && (M % 256) == 0 && (N % 256) == 0 && (bn_hint == 512 || bn == 256);
    if (bn_hint == 512 && !eligible) return cudaErrorInvalidValue;
    // (forwards of a few thousand rows gain nothing from pairs; measured at 4608 rows: 3 to 5 % slower)
    if (eligible && (bn_hint == 512 || (pair_on && splits == 1 && (M >= 8192 || pair_any_size) && mt * (N / 256) > 2 * SMS))) {
      CUtensorMap mb_half;
      if ((e = get_tensor_map(W, N, K, K, 128, BK, &mb_half)) != cudaSuccess) return e;
      const int tiles_m2 = M / 256, tiles_n = N / 256;
      const long long tiles = (long long)tiles_m2 * tiles_n;
      const unsigned pairs = (unsigned)(tiles < SMS / 2 ? tiles : SMS / 2);
      launch_k(gemm_tc_pair_kernel, dim3(2 * pairs), dim3(PAIR_THREADS), (size_t)PAIR_SMEM, st, ma, mb_half, mo, tma_out, M, N, K, epi,
               bias, out, ldc, status, qd, skip, tiles_m2, tiles_n, (long long)N * K * 2 <= (48ll << 20) ? 1 : 0);
      return cudaGetLastError();
    }
  }
  // many 256-wide tiles and no K split: the persistent kernel (SDD_GEMM_PERSIST=0 switches it off)
  static const bool persist_on = [] { const char* e = getenv("SDD_GEMM_PERSIST"); return e == nullptr || atoi(e) != 0; }();
  if (persist_on && bn == 256 && splits == 1 && mt * ((N + 255) / 256) > 2 * SMS) {
    const HeadStats hs = stats_for((N + 255) / 256);
    if (hilo)
      return launch_persist<256, true>(ma, mb, ml, mo, tma_out, M, N, K, epi, bias, out, out_lo, ldc, status, st, qd, skip, hs);
    return launch_persist<256, false>(ma, mb, ml, mo, tma_out, M, N, K, epi, bias, out, out_lo, ldc, status, st, qd, skip, hs);
  }
  switch (bn) {
    case 256: return launch_hl<256, false>(hilo, ma, mb, ml, mo, tma_out, M, N, K, epi, bias, out, out_lo, ldc, status, st, qd, splits, skip);
    case 128: return launch_hl<128, false>(hilo, ma, mb, ml, mo, tma_out, M, N, K, epi, bias, out, out_lo, ldc, status, st, qd, splits, skip);
    case 64: return launch_hl<64, false>(hilo, ma, mb, ml, mo, tma_out, M, N, K, epi, bias, out, out_lo, ldc, status, st, qd, splits, skip);
    default: return launch_hl<32, false>(hilo, ma, mb, ml, mo, tma_out, M, N, K, epi, bias, out, out_lo, ldc, status, st, qd, splits, skip);
  }
}

}  // namespace sdd
