// Tensor-core attention for sm_100a (bf16 in, fp32 soft-max state), d_head = 64.
//
// One CTA owns 128 query rows of one head of one sequence and walks over the keys in tiles of 128:
//   S  = Q K^T          tcgen05.mma, 128 x 128 fp32 accumulator in TMEM (Q, K tiles via TMA, K-major)
//   P  = exp2(S - m)    eight soft-max warps, two threads per query row (tcgen05.ld gives a thread its row), each an
//                       independent online soft-max over its 64 keys of the tile with its own reference maximum m;
//                       P is written as bf16 into shared memory in the 128-byte-swizzled K-major layout
//   PV = P V            tcgen05.mma with V^T tiles ([d_head, keys], keys contiguous) as the second operand; one
//                       64-column fp32 accumulator per half of the key tile, accumulating over the tiles in TMEM and
//                       rescaled there (tcgen05.ld / st) when a thread moves its reference maximum.
// The same kernel serves the drafter (no mask: every row sees every row of its sequence) and the target
// (row at position p sees cache positions 0..p).  V is consumed transposed, which the QKV GEMM's epilogue
// produces for free; that keeps both MMAs on K-major operands.
// Shared memory: the K tile of a stage is dead once S = Q K^T has completed and stays unused until P V has
// completed (only then is the stage handed back to the producer), so the first half of P (keys 0..63) is written
// over it; with that the CTA needs 96 KB and two CTAs share an SM, one's soft-max overlapping the other's MMAs.
// PIPE variant (grids of at most one CTA per SM, where a CTA's chain of key tiles is what bounds the launch): S is
// double-buffered in TMEM (512 columns, one CTA per SM) and the K / V^T ring has three stages, so S(t+1) = Q K(t+1)^T is
// issued before the MMA thread waits for P(t) and is complete when the soft-max warps get to it; a tile's chain is then
// soft-max -> next soft-max instead of S -> soft-max -> P V -> S.  The second half of P has two buffers there (the
// first half lies over the tile's own K stage), so P(t+1) is written while P(t) V(t) may still be running.
// Waits are bounded exactly as in the GEMM kernel.
#include <cstdlib>
#include <mutex>
#include <type_traits>

#include "sdd_kernels.h"
#include "sdd_tc.cuh"

namespace sdd {
namespace tc {

constexpr int AT_THREADS = 320;              // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..9: soft-max
constexpr int AT_DH = 64;
constexpr int AT_Q_BYTES = 128 * 64 * 2;            // 16 KB
constexpr int AT_P_BYTES = 128 * 64 * 2;            // P k-block 1 (keys 64..127); k-block 0 reuses the K tile, see below
constexpr int AT_K_BYTES = 128 * 64 * 2;            // 16 KB
constexpr int AT_VT_BYTES = 2 * 64 * 64 * 2;        // two boxes [64 d_head rows x 64 keys]: 16 KB
constexpr int AT_STAGE_BYTES = AT_K_BYTES + AT_VT_BYTES;
// PIPE = false: two K / V^T stages, 96 KB, two CTAs per SM; TMEM: S in columns 0..127, PV accumulators 128..191 and 192..255
// PIPE = true : three stages and two buffers for the second half of P, 144 KB, one CTA per SM; TMEM: S buffers 0..127 and
//               128..255, PV accumulators 256..319 and 320..383
template <bool PIPE> constexpr int at_stages() { return PIPE ? 3 : 2; }
template <bool PIPE> constexpr int at_p_bytes() { return (PIPE ? 2 : 1) * AT_P_BYTES; }   // PIPE: P k-block 1 double-buffered
template <bool PIPE> constexpr int at_bar_off() { return AT_Q_BYTES + at_p_bytes<PIPE>() + at_stages<PIPE>() * AT_STAGE_BYTES; }
template <bool PIPE> constexpr int at_smem() { return at_bar_off<PIPE>() + 1024 + 128 + 3 * 1024; }   // barriers, then the soft-max exchange arrays
template <bool PIPE> constexpr uint32_t at_tmem_cols() { return PIPE ? 512u : 256u; }
template <bool PIPE> constexpr uint32_t at_acc_col() { return PIPE ? 256u : 128u; }
// key-split launches add a receive area for the other CTAs' partial states (it must not lie over tiles that this CTA
// may still be using when a faster CTA sends): at most 136 rows of 64 floats plus their m and l
template <bool PIPE> constexpr int at_recv_off() { return at_bar_off<PIPE>() + 3328; }
template <bool PIPE> constexpr int at_smem_split() { return at_recv_off<PIPE>() + 36 * 1024 + 1024; }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct AttnParams {
  __nv_bfloat16* out;
  int ld_out;
  const int* ctx_len;
  int mode;             // 0: drafter, no mask; 1: target verify (position c-1+i); 2: target prefill (position i)
  int gamma;
  int q_rows_per_seq;   // rows of one sequence in the Q tensor and in out
  int k_rows_per_seq;   // rows of one sequence in the K tensor
  int q_col0, k_col0;   // column of head 0 in the Q / K tensors
  int d;                // model width = rows of one sequence in the V^T tensor
  int* status;
  const int* skip;      // may be null; *skip != 0: return at once (skipped drafter evaluation)
  int kv_split;         // > 1 (unmasked mode, small grids): a cluster of kv_split CTAs shares the key tiles of one query
                        // tile (CTA r takes tiles r, r + kv_split, ...); the partial soft-max states are merged row slice by
                        // row slice, one slice per CTA
};

// stores into the shared memory of another CTA of the cluster (address from map_to_cta); they complete asynchronously
// and are visible to that CTA after the next cluster barrier
__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

template <bool PIPE>
__global__ void __launch_bounds__(AT_THREADS, PIPE ? 1 : 2)
attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_vt, const AttnParams prm) {
  constexpr int AT_KV_STAGES = at_stages<PIPE>();
  constexpr int AT_BAR_OFF = at_bar_off<PIPE>();
  constexpr int AT_RECV_OFF = at_recv_off<PIPE>();
  constexpr uint32_t AT_TMEM_COLS = at_tmem_cols<PIPE>();
  constexpr uint32_t ACC_COL = at_acc_col<PIPE>();
  constexpr int P_TOTAL = at_p_bytes<PIPE>();
  const int kv_split = prm.kv_split, kv_rank = (int)blockIdx.x % kv_split;   // cluster = kv_split consecutive CTAs in x
  const int qt = (int)blockIdx.x / kv_split, h = blockIdx.y, b = blockIdx.z;

  // set-up that touches only shared and tensor memory comes first: it runs under the tail of the kernel ahead
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base;
  auto sP = [&](int t) { return base + AT_Q_BYTES + (PIPE ? (uint32_t)(t & 1) * AT_P_BYTES : 0u); };   // P k-block 1 of tile t
  auto sK = [&](int s) { return base + AT_Q_BYTES + P_TOTAL + s * AT_STAGE_BYTES; };
  auto sVT = [&](int s) { return sK(s) + AT_K_BYTES; };
  const uint32_t bars = base + AT_BAR_OFF;
  // PIPE keeps one barrier per parity of the tile for "P written", "P V done" and "S done": a soft-max warp may be one
  // tile ahead of the slowest one there (S(t+1) is complete before the last warp has finished tile t), so its arrivals
  // for tile t + 1 must not be counted with those still missing for tile t; !PIPE uses only the barriers [0]
  const uint32_t q_full = bars;
  auto p_ready = [&](int i) { return bars + 8 + 8u * i; };
  auto pv_full = [&](int i) { return bars + 24 + 8u * i; };
  auto s_full = [&](int i) { return bars + 40 + 8u * i; };
  auto kv_full = [&](int s) { return bars + 56 + 8u * s; };
  auto kv_empty = [&](int s) { return bars + 80 + 8u * s; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + AT_BAR_OFF + 104);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + AT_BAR_OFF + 112);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < 2; ++i) { mbar_init(p_ready(i), 256); mbar_init(pv_full(i), 1); mbar_init(s_full(i), 1); }
    for (int s = 0; s < AT_KV_STAGES; ++s) { mbar_init(kv_full(s), 1); mbar_init(kv_empty(s), 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(tmem_slot, AT_TMEM_COLS);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  pdl_launch_dependents();
  pdl_wait();   // ctx_len and Q / K / V^T come from earlier kernels
  // The Q tile and the first K / V^T tile go out at once: their coordinates do not depend on the context length or the
  // skip flag, whose loads would otherwise sit in front of them (with a key split the first tile of a CTA may not exist,
  // so only unsplit launches do this).  A CTA that turns out to have nothing to do waits for the copies and drops them.
  const bool spec = kv_split == 1;
  if (spec && threadIdx.x == 0) {
    mbar_expect_tx(q_full, AT_Q_BYTES);
    tma_load_2d(sQ, &map_q, q_full, prm.q_col0 + h * AT_DH, b * prm.q_rows_per_seq + qt * 128);
    mbar_expect_tx(kv_full(0), AT_STAGE_BYTES);
    tma_load_2d(sK(0), &map_k, kv_full(0), prm.k_col0 + h * AT_DH, b * prm.k_rows_per_seq);
    tma_load_2d(sVT(0), &map_vt, kv_full(0), 0, b * prm.d + h * AT_DH);
    tma_load_2d(sVT(0) + 64 * 64 * 2, &map_vt, kv_full(0), 64, b * prm.d + h * AT_DH);
  }
  // a skipped drafter evaluation, or a tile of padding rows only: nothing to do (uniform over the CTA and its cluster)
  bool active = !(prm.skip != nullptr && *prm.skip);
  const int c = active ? prm.ctx_len[b] : 1;
  const int q0 = qt * 128;
  int n_valid_q;
  if (prm.mode == 0) n_valid_q = c + prm.gamma;
  else if (prm.mode == 1) n_valid_q = prm.q_rows_per_seq;
  else n_valid_q = c - 1;
  if (n_valid_q > prm.q_rows_per_seq) n_valid_q = prm.q_rows_per_seq;
  if (q0 >= n_valid_q) active = false;
  const int last_valid = (n_valid_q < q0 + 128 ? n_valid_q : q0 + 128) - 1;
  int n_keys_cta;
  if (prm.mode == 0) n_keys_cta = c + prm.gamma;
  else if (prm.mode == 1) n_keys_cta = c - 1 + last_valid + 1;
  else n_keys_cta = last_valid + 1;
  if (n_keys_cta > prm.k_rows_per_seq) n_keys_cta = prm.k_rows_per_seq;
  const int num_kt = active ? (n_keys_cta + 127) / 128 : 0;
  const int my_kt = kv_rank < num_kt ? (num_kt - kv_rank + kv_split - 1) / kv_split : 0;   // key tiles of this CTA
  // completion of P(t) V(t): PIPE keeps one barrier per parity of t, so that a wait for tile t - 2 cannot be taken for
  // one on a phase still to come
  auto wait_pv = [&](int t) {
    return mbar_wait(pv_full(PIPE ? (t & 1) : 0), (uint32_t)(PIPE ? (t >> 1) : t) & 1u, abort_flag, prm.status);
  };

  if (!active) {
    if (spec && threadIdx.x == 0) {   // the copies issued ahead must have landed before the shared memory is given back
      long long t0 = clock64();
      while (!mbar_try(q_full, 0u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
      t0 = clock64();
      while (!mbar_try(kv_full(0), 0u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
    }
  } else if (warp == 0) {
    if (lane == 0 && my_kt > 0) {   // (an unsplit launch that is active has at least one key tile)
      if (!spec) {
        mbar_expect_tx(q_full, AT_Q_BYTES);
        tma_load_2d(sQ, &map_q, q_full, prm.q_col0 + h * AT_DH, b * prm.q_rows_per_seq + q0);
      }
      int issued = spec ? 1 : 0;
      for (int it = issued; it < my_kt; ++it) {
        const int t = kv_rank + it * kv_split;      // key tile; `it` counts this CTA's iterations (stages, phases)
        const int s = it % AT_KV_STAGES;
        if (!mbar_wait(kv_empty(s), ((uint32_t)(it / AT_KV_STAGES) & 1u) ^ 1u, abort_flag, prm.status)) break;
        mbar_expect_tx(kv_full(s), AT_STAGE_BYTES);
        tma_load_2d(sK(s), &map_k, kv_full(s), prm.k_col0 + h * AT_DH, b * prm.k_rows_per_seq + t * 128);
        tma_load_2d(sVT(s), &map_vt, kv_full(s), t * 128, b * prm.d + h * AT_DH);
        tma_load_2d(sVT(s) + 64 * 64 * 2, &map_vt, kv_full(s), t * 128 + 64, b * prm.d + h * AT_DH);
        issued = it + 1;
      }
      if (*abort_flag) {   // do not leave while copies into this CTA's shared memory may be in flight
        long long t0 = clock64();
        while (!mbar_try(q_full, 0u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        for (int t = issued > AT_KV_STAGES ? issued - AT_KV_STAGES : 0; t < issued; ++t) {
          t0 = clock64();
          while (!mbar_try(kv_full(t % AT_KV_STAGES), (uint32_t)(t / AT_KV_STAGES) & 1u) && clock64() - t0 < WAIT_LIMIT_CYCLES) {}
        }
      }
    }
    if (kv_split > 1) { __syncwarp(); cluster_sync_all(); }   // see the soft-max warps
  } else if (warp == 1) {
    if (lane == 0 && my_kt > 0) {
      constexpr uint32_t idesc_s = make_idesc<128>();
      constexpr uint32_t idesc_pv = make_idesc<64>();
      bool ok = mbar_wait(q_full, 0u, abort_flag, prm.status);
      const uint64_t dq = make_smem_desc(sQ);
      // S(t) = Q K(t)^T into S buffer t & 1 (PIPE) or the one S buffer; t counts this CTA's iterations
      auto issue_s = [&](int t) -> bool {
        const int s = t % AT_KV_STAGES;
        if (!mbar_wait(kv_full(s), (uint32_t)(t / AT_KV_STAGES) & 1u, abort_flag, prm.status)) return false;
        fence_after_sync();
        const uint64_t dk = make_smem_desc(sK(s));
        const uint32_t sc = PIPE ? (uint32_t)(t & 1) * 128u : 0u;
#pragma unroll
        for (int k = 0; k < 4; ++k) umma(tmem_base + sc, dq + 2u * k, dk + 2u * k, idesc_s, k > 0 ? 1u : 0u);
        umma_commit(s_full(PIPE ? (t & 1) : 0));
        return true;
      };
      if (PIPE && ok) ok = issue_s(0);
      for (int t = 0; t < my_kt && ok; ++t) {        // t: this CTA's iteration (the key tile does not matter here)
        const int s = t % AT_KV_STAGES;
        if (PIPE) {
          // the next tile's scores are issued before the wait for this tile's probabilities: the soft-max warps are done
          // with S buffer (t + 1) & 1 since p_ready(t - 1), which this thread has seen
          if (t + 1 < my_kt) ok = issue_s(t + 1);
        } else {
          ok = issue_s(t);
        }
        if (!ok) break;
        ok = mbar_wait(p_ready(PIPE ? (t & 1) : 0), (uint32_t)(PIPE ? (t >> 1) : t) & 1u, abort_flag, prm.status);
        if (!ok) break;
        fence_after_sync();
        // one accumulator per half of the key tile (keys 0..63 and keys 64..127 of the tile); both add up over the
        // CTA's tiles in TMEM
#pragma unroll
        for (int kb = 0; kb < 2; ++kb) {
          const uint64_t dp = make_smem_desc(kb == 0 ? sK(s) : sP(t));
          const uint64_t dv = make_smem_desc(sVT(s) + kb * (64 * 64 * 2));
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma(tmem_base + ACC_COL + (uint32_t)(kb * 64), dp + 2u * k, dv + 2u * k, idesc_pv, (t | k) ? 1u : 0u);
        }
        umma_commit(pv_full(PIPE ? (t & 1) : 0));
        umma_commit(kv_empty(s));
      }
    }
    if (kv_split > 1) { __syncwarp(); cluster_sync_all(); }
  } else {
    // soft-max warps 2..9: two threads per query row.  Warp w reads TMEM lane quarter w & 3; warps 2..5 take key
    // columns 0..63 of the tile (and output columns 0..31), warps 6..9 key columns 64..127 (output columns 32..63).
    const int hf = (warp - 2) >> 2;
    const int r = (warp & 3) * 32 + lane;
    const int i = q0 + r;
    const bool valid = i < n_valid_q;
    int key_limit;                                     // keys [0, key_limit) are visible to this row
    if (prm.mode == 0) key_limit = n_keys_cta;
    else if (prm.mode == 1) key_limit = c - 1 + i + 1;
    else key_limit = i + 1;
    if (key_limit > n_keys_cta) key_limit = n_keys_cta;
    if (!valid) key_limit = 0;
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16);
    const float scale = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) * log2(e)
    float* s_max = reinterpret_cast<float*>(gbase + AT_BAR_OFF + 128);          // [2 tile parities][2 halves][128 rows]
    float* s_l = s_max + 2 * 2 * 128;                                            // [2 halves][128 rows]
    float m = -INFINITY, l = 0.f;
    const int sw = r & 7;
    bool ok = true;
    // The two threads of a row are independent online soft-maxes over "their" 64 keys of every tile: own reference
    // maximum m, own sum l, own accumulator in TMEM (P_half x V_half).  The accumulator is rescaled in place, and only
    // when the thread's maximum has grown by more than 2^8 since its reference was set (the probabilities are then
    // bounded by 256, exact arithmetic otherwise unchanged), so the common tile has no fold, no exchange between the
    // halves and no barrier among the warps.  The halves are combined once, after the last tile.
    const uint32_t t_acc = t_lane + ACC_COL + (uint32_t)(hf * 64);
    uint32_t v[32];
    for (int it = 0; it < my_kt; ++it) {
      const int t = kv_rank + it * kv_split;           // key tile; `it` counts this CTA's iterations (stages, phases)
      ok = __all_sync(0xffffffffu, mbar_wait(s_full(PIPE ? (it & 1) : 0), (uint32_t)(PIPE ? (it >> 1) : it) & 1u, abort_flag,
                                             prm.status));
      if (!ok) break;
      fence_after_sync();
      const int key0 = t * 128 + hf * 64;
      const uint32_t t_s = t_lane + (PIPE ? (uint32_t)(it & 1) * 128u : 0u);    // this tile's S buffer
      // this thread's 64 probabilities are one row of a P k-block: block 0 lies over the stage's (consumed) K tile
      uint8_t* p_row = gbase + (hf == 0 ? AT_Q_BYTES + P_TOTAL + (it % AT_KV_STAGES) * AT_STAGE_BYTES
                                        : AT_Q_BYTES + (PIPE ? (it & 1) * AT_P_BYTES : 0)) + r * 128;
      // tcgen05.ld / st are warp-collective: every branch around them is taken by whole warps
      const bool full_w = __all_sync(0xffffffffu, key0 + 64 <= key_limit);
      // !PIPE: the 64 scores are read twice from TMEM (once for the maximum, once for the exponentials) instead of being
      // kept in 64 registers: two CTAs per SM need the kernel to stay below 100 registers.  PIPE (one CTA per SM) keeps them.
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains
      auto max_chunk = [&](const uint32_t (&x)[32], int cc) {
        if (full_w) {
#pragma unroll
          for (int j = 0; j < 32; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], __uint_as_float(x[j]));
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (key0 + cc * 32 + j < key_limit) mx4[j & 3] = fmaxf(mx4[j & 3], __uint_as_float(x[j]));
        }
      };
      uint32_t sc[PIPE ? 2 : 1][32];
      if constexpr (PIPE) {
        tmem_ld32_issue(t_s + (uint32_t)(hf * 64), sc[0]);
        tmem_ld32_issue(t_s + (uint32_t)(hf * 64 + 32), sc[1]);
        tmem_ld_wait(sc[0], sc[1]);
        max_chunk(sc[0], 0);
        max_chunk(sc[1], 1);
      } else {
#pragma unroll 1
        for (int cc = 0; cc < 2; ++cc) {
          tmem_ld32(t_s + (uint32_t)(hf * 64 + cc * 32), v);
          max_chunk(v, cc);
        }
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale;     // -inf: no visible key
      if (__any_sync(0xffffffffu, mx > m + 8.f)) {
        // new reference for every lane of the warp (exact maximum); the accumulator and the sum follow it
        const float m_new = fmaxf(m, mx);
        const float corr = (m == -INFINITY || m_new == -INFINITY) ? 0.f : ex2(m - m_new);
        if (it > 0) {
          ok = __all_sync(0xffffffffu, wait_pv(it - 1));
          if (!ok) break;
          fence_after_sync();
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            tmem_ld32(t_acc + (uint32_t)(hh * 32), v);
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * corr);
            tmem_st32(t_acc + (uint32_t)(hh * 32), v);
          }
        }
        l *= corr;
        m = m_new;
      }
      // P(t) overwrites the buffer of P(t-1) (PIPE: of P(t-2)) once that tile's P V has read it
      if (it >= (PIPE ? 2 : 1)) {
        ok = __all_sync(0xffffffffu, wait_pv(it - (PIPE ? 2 : 1)));
        if (!ok) break;
      }
      const float m_use = m == -INFINITY ? 0.f : m;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      auto exp_chunk = [&](auto full_tag, auto cc_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        constexpr int cc = decltype(cc_tag)::value;
        if constexpr (!PIPE) tmem_ld32(t_s + (uint32_t)(hf * 64 + cc * 32), v);
        const uint32_t (&x)[32] = PIPE ? sc[PIPE ? cc : 0] : v;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int j0 = g * 8 + 2 * e;
            float p0 = ex2(fmaf(__uint_as_float(x[j0]), scale, -m_use));
            float p1 = ex2(fmaf(__uint_as_float(x[j0 + 1]), scale, -m_use));
            if (!FULL) {
              if (!(key0 + cc * 32 + j0 < key_limit)) p0 = 0.f;
              if (!(key0 + cc * 32 + j0 + 1 < key_limit)) p1 = 0.f;
            }
            sum4[e] += p0 + p1;
            __nv_bfloat162 h2 = __floats2bfloat162_rn(p0, p1);
            pk[e] = *reinterpret_cast<uint32_t*>(&h2);
          }
          *reinterpret_cast<uint4*>(p_row + (((cc * 4 + g) ^ sw) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      };
      // two copies, chosen by a real (warp-uniform) branch: the visibility tests cost a third of the issue slots when
      // they are predicated into the common unmasked path
      using C0 = std::integral_constant<int, 0>;
      using C1 = std::integral_constant<int, 1>;
      if (full_w) { exp_chunk(std::true_type{}, C0{}); exp_chunk(std::true_type{}, C1{}); }
      else { exp_chunk(std::false_type{}, C0{}); exp_chunk(std::false_type{}, C1{}); }
      l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      fence_before_sync();          // accumulator reads / writes above are ordered before the MMA that follows the arrive
      fence_async_smem();
      mbar_arrive(p_ready(PIPE ? (it & 1) : 0));
    }
    if (ok && my_kt > 0) ok = __all_sync(0xffffffffu, wait_pv(my_kt - 1));
    ok = named_bar_and(1, 256, ok);
    float o[AT_DH / 2];                                // this thread's 32 output columns (unnormalised)
#pragma unroll
    for (int j = 0; j < AT_DH / 2; ++j) o[j] = 0.f;
    if (ok) {
      // combine the two halves of every row: common maximum, weights, sum; this thread's 32 output columns from both
      // halves' accumulators
      fence_after_sync();
      float* s_m = s_max;                              // [2 halves][128 rows]
      s_m[hf * 128 + r] = m;
      s_l[hf * 128 + r] = l;
      named_bar_sync(2, 256);
      const float m_o = s_m[(hf ^ 1) * 128 + r], l_o = s_l[(hf ^ 1) * 128 + r];
      const float mm = fmaxf(m, m_o);
      const float w_me = m == -INFINITY ? 0.f : ex2(m - mm), w_o = m_o == -INFINITY ? 0.f : ex2(m_o - mm);
      l = l * w_me + l_o * w_o;
      m = mm;
      if (my_kt > 0) {
        tmem_ld32(t_lane + ACC_COL + (uint32_t)(hf * 64 + hf * 32), v);        // own half's accumulator
#pragma unroll
        for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(v[j]) * w_me;
        tmem_ld32(t_lane + ACC_COL + (uint32_t)((hf ^ 1) * 64 + hf * 32), v);  // the other half's
#pragma unroll
        for (int j = 0; j < 32; ++j) o[j] = fmaf(__uint_as_float(v[j]), w_o, o[j]);
      }
    }
    bool writes_row = kv_split == 1;
    if (kv_split > 1) {
      // Merge of the cluster's partial soft-max states (m, l, o).  The 128 rows are dealt out to the CTAs in slices of
      // sz rows; every thread sends its row's state to the CTA that owns the row (asynchronous remote stores into the
      // receive area behind the kernel's other shared memory), one cluster barrier, then the owner's thread of
      // that row adds up what it received.  recv_o[src][row in slice][64], recv_m / recv_l[src][row in slice].
      const int sz = (128 + kv_split - 1) / kv_split;
      const int owner = r / sz, rloc = r - owner * sz;
      float* recv_o = reinterpret_cast<float*>(gbase + AT_RECV_OFF);
      float* recv_m = recv_o + kv_split * sz * AT_DH;
      float* recv_l = recv_m + kv_split * sz;
      const bool have = ok && my_kt > 0;
      if (owner != kv_rank) {
        const int slot = kv_rank * sz + rloc;
        if (hf == 0) {
          st_cluster_f32(map_to_cta(smem_u32(recv_m + slot), (uint32_t)owner), have ? m : -INFINITY);
          st_cluster_f32(map_to_cta(smem_u32(recv_l + slot), (uint32_t)owner), l);
        }
        if (have) {
          const uint32_t dst = map_to_cta(smem_u32(recv_o + slot * AT_DH + hf * 32), (uint32_t)owner);
#pragma unroll
          for (int j = 0; j < 8; ++j) st_cluster_v4(dst + 16u * j, o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
        }
      }
      cluster_sync_all();
      if (owner == kv_rank && ok) {
        writes_row = true;
        float mx = have ? m : -INFINITY;
        for (int p = 0; p < kv_split; ++p)
          if (p != kv_rank) mx = fmaxf(mx, recv_m[p * sz + rloc]);
        const float w0 = (have && m != -INFINITY) ? ex2(m - mx) : 0.f;
        l *= w0;
#pragma unroll
        for (int j = 0; j < AT_DH / 2; ++j) o[j] *= w0;
        for (int p = 0; p < kv_split; ++p) {
          if (p == kv_rank) continue;
          const float mp = recv_m[p * sz + rloc];
          if (mp == -INFINITY) continue;               // that CTA had no key tile (or no visible key) for this row
          const float wp = ex2(mp - mx);
          l = fmaf(recv_l[p * sz + rloc], wp, l);
          const float4* src = reinterpret_cast<const float4*>(recv_o + (p * sz + rloc) * AT_DH + hf * 32);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float4 x = src[j];
            o[4 * j] = fmaf(x.x, wp, o[4 * j]); o[4 * j + 1] = fmaf(x.y, wp, o[4 * j + 1]);
            o[4 * j + 2] = fmaf(x.z, wp, o[4 * j + 2]); o[4 * j + 3] = fmaf(x.w, wp, o[4 * j + 3]);
          }
        }
      }
    }
    if (ok && writes_row) {
      if (valid) {
        const float inv = 1.f / l;
        __nv_bfloat16* dst = prm.out + ((long long)b * prm.q_rows_per_seq + i) * prm.ld_out + h * AT_DH + hf * 32;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 h2 = __floats2bfloat162_rn(o[g * 8 + 2 * e] * inv, o[g * 8 + 2 * e + 1] * inv);
            pk[e] = *reinterpret_cast<uint32_t*>(&h2);
          }
          *reinterpret_cast<uint4*>(dst + g * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    fence_after_sync();
    tmem_dealloc(tmem_base, AT_TMEM_COLS);
  }
}

}  // namespace tc

cudaError_t tc_prepare_attn() {
  cudaError_t e = cudaFuncSetAttribute(tc::attn_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::at_smem_split<false>());
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(tc::attn_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::at_smem_split<true>());
}

cudaError_t launch_attn_tc(const __nv_bfloat16* q, long long q_rows_total, int q_ld, int q_col0, const __nv_bfloat16* k,
                           long long k_rows_total, int k_ld, int k_col0, int k_rows_per_seq, const __nv_bfloat16* vt,
                           int vt_ld, __nv_bfloat16* out, int ld_out, const int* ctx_len, int batch, int n_head, int d,
                           int gamma, int mode, int q_rows_per_seq, int* status, cudaStream_t st, const int* skip) {
  using namespace tc;
  if (q_rows_per_seq <= 0) return cudaSuccess;
  if (d != n_head * AT_DH || (ld_out & 7) != 0) return cudaErrorInvalidValue;
  CUtensorMap mq, mk, mv;
  cudaError_t e;
  if ((e = get_tensor_map(q, q_rows_total, q_ld, q_ld, 128, 64, &mq)) != cudaSuccess) return e;
  if ((e = get_tensor_map(k, k_rows_total, k_ld, k_ld, 128, 64, &mk)) != cudaSuccess) return e;
  if ((e = get_tensor_map(vt, (long long)batch * d, vt_ld, vt_ld, 64, 64, &mv)) != cudaSuccess) return e;
  static std::once_flag once;
  static cudaError_t prep = cudaSuccess;
  std::call_once(once, [] { prep = tc_prepare_attn(); });
  if (prep != cudaSuccess) return prep;
  AttnParams p;
  p.out = out; p.ld_out = ld_out; p.ctx_len = ctx_len; p.mode = mode; p.gamma = gamma;
  p.q_rows_per_seq = q_rows_per_seq; p.k_rows_per_seq = k_rows_per_seq; p.q_col0 = q_col0; p.k_col0 = k_col0;
  p.d = d; p.status = status; p.skip = skip; p.kv_split = 1;
  dim3 grid((q_rows_per_seq + 127) / 128, n_head, batch);
  // at most one CTA per SM: the launch is bound by each CTA's chain of key tiles, not by throughput -> PIPE variant
  // (SDD_ATTN_PIPE=0 switches it off)
  static const bool pipe_on = [] { const char* e = getenv("SDD_ATTN_PIPE"); return e == nullptr || atoi(e) != 0; }();
  const bool pipe = pipe_on && (long long)grid.x * grid.y * grid.z <= 148;
  // Unmasked attention on a grid that leaves most SMs idle (one sequence): the key tiles of a query tile are shared out
  // over a cluster of CTAs, which shortens the chain of dependent tiles per CTA; CTA 0 merges the partial states.
  // SDD_ATTN_SPLIT=0 switches it off.
  if (mode == 0) {
    const char* e = getenv("SDD_ATTN_SPLIT");
    const long long ctas = (long long)grid.x * grid.y * grid.z;
    int split = (q_rows_per_seq + 127) / 128;
    if (split > 8) split = 8;
    // only when every CTA gets exactly one key tile and the grid fits one CTA per SM (with the receive area): with
    // uneven shares the longest chain is as long as before and the merge only adds to it (measured over a whole
    // generation: 5.18 ms per round without any split, 5.36 ms with partial splits)
    if (ctas * split > 148) split = 1;
    if ((e == nullptr || atoi(e) != 0) && split > 1) {
      p.kv_split = split;
      grid.x *= split;
      launch_k_cluster(attn_tc_kernel<false>, grid, dim3(AT_THREADS), at_smem_split<false>(), st, (unsigned)split, mq, mk, mv, p);
      return cudaGetLastError();
    }
  }
  if (pipe) launch_k(attn_tc_kernel<true>, dim3(grid), dim3(AT_THREADS), at_smem<true>(), st, mq, mk, mv, p);
  else launch_k(attn_tc_kernel<false>, dim3(grid), dim3(AT_THREADS), at_smem<false>(), st, mq, mk, mv, p);
  return cudaGetLastError();
}

}  // namespace sdd
