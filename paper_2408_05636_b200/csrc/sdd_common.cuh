// Shared device/host helpers of the SpecDiff CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/sdd.h"

namespace sdd {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11) and the random streams of a round.
//   counter = (c0, slot j, round r, purpose << 24 | step k << 16 | sequence b)
//   per-vocabulary streams: c0 = v >> 2, element v takes word v & 3; scalar streams: c0 = 0, word 0
// ---------------------------------------------------------------------------------------------
enum : uint32_t { RNG_UNMASK = 1, RNG_DRAFT = 2, RNG_ACCEPT = 3, RNG_RESID = 4, RNG_BONUS = 5 };

struct PhiloxKey {
  uint32_t k0, k1;
};

__host__ __device__ inline PhiloxKey make_key(uint64_t seed) {
  PhiloxKey k;
  k.k0 = (uint32_t)(seed & 0xFFFFFFFFull);
  k.k1 = (uint32_t)(seed >> 32);
  return k;
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, PhiloxKey key) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t k0 = key.k0, k1 = key.k1;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += W0; k1 += W1;
  }
  return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint32_t rng_c3(uint32_t purpose, uint32_t k, uint32_t b) {
  return (purpose << 24) | (k << 16) | b;
}

// ((w >> 9) + 0.5) * 2^-23 : an odd multiple of 2^-24, exact in fp32, strictly inside (0, 1)
__device__ __forceinline__ float word_to_uniform(uint32_t w) {
  return (float)(((w >> 9) << 1) | 1u) * 5.9604644775390625e-08f;
}

__device__ __forceinline__ float scalar_uniform(PhiloxKey key, uint32_t purpose, uint32_t rnd, uint32_t k, uint32_t j,
                                                uint32_t b) {
  return word_to_uniform(philox4x32_10(0u, j, rnd, rng_c3(purpose, k, b), key).x);
}

// Gumbel variate -log(-log u) for u = odd multiple of 2^-24 in (0, 1), to about 2e-6 absolute.
// The inner logarithm needs care next to u = 1, where the largest variates (the likely arg-max winners) come
// from: there 1 - u is exact in fp32 and -log(1 - t) is summed as a series; elsewhere the hardware log2 does.
__device__ __forceinline__ float gumbel_from_uniform(float u) {
  const float t = 1.0f - u;
  float ser = fmaf(t, 1.f / 9.f, 1.f / 8.f);
  ser = fmaf(t, ser, 1.f / 7.f);
  ser = fmaf(t, ser, 1.f / 6.f);
  ser = fmaf(t, ser, 1.f / 5.f);
  ser = fmaf(t, ser, 1.f / 4.f);
  ser = fmaf(t, ser, 1.f / 3.f);
  ser = fmaf(t, ser, 1.f / 2.f);
  ser = fmaf(t, ser, 1.f);
  const float y = t < 0.125f ? t * ser : -__logf(u);
  return -__logf(y);
}

// ---------------------------------------------------------------------------------------------
// reductions
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// (score, index) arg-max; ties go to the lowest index
struct ArgMax {
  float s;
  int i;
};
__device__ __forceinline__ ArgMax argmax_better(ArgMax a, ArgMax b) {
  return (b.s > a.s || (b.s == a.s && b.i < a.i)) ? b : a;
}
__device__ __forceinline__ ArgMax warp_argmax(ArgMax a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ArgMax b;
    b.s = __shfl_xor_sync(0xffffffffu, a.s, o);
    b.i = __shfl_xor_sync(0xffffffffu, a.i, o);
    a = argmax_better(a, b);
  }
  return a;
}

// online soft-max accumulator: sum of exp(z - m)
struct MaxSum {
  float m, s;
};
__device__ __forceinline__ MaxSum maxsum_merge(MaxSum a, MaxSum b) {
  const float m = fmaxf(a.m, b.m);
  MaxSum r;
  r.m = m;
  r.s = (a.m == -INFINITY ? 0.f : a.s * __expf(a.m - m)) + (b.m == -INFINITY ? 0.f : b.s * __expf(b.m - m));
  return r;
}
__device__ __forceinline__ MaxSum warp_maxsum(MaxSum a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    MaxSum b;
    b.m = __shfl_xor_sync(0xffffffffu, a.m, o);
    b.s = __shfl_xor_sync(0xffffffffu, a.s, o);
    a = maxsum_merge(a, b);
  }
  return a;
}

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float gelu_tanh(float x) {
  const float c = 0.7978845608028654f;  // sqrt(2/pi)
  return 0.5f * x * (1.f + tanhf(c * (x + 0.044715f * x * x * x)));
}

// ---------------------------------------------------------------------------------------------
// programmatic dependent launch: a kernel launched with the attribute may start (and run its
// prologue) while its predecessor in the stream drains; pdl_wait() blocks until the predecessor has
// completed and its writes are visible.  Every kernel of the library calls pdl_wait() before its
// first access to global memory, so stream order is preserved transitively.  Without the launch
// attribute the instruction does nothing.
// pdl_launch_dependents() comes BEFORE the wait: the next kernel's CTAs become resident (barriers, tensor-memory
// allocation, descriptor and weight prefetch) while this kernel is still waiting for its own predecessor, so a chain
// of short kernels runs two or three launches ahead.  Two rules keep that safe.  (1) A kernel that allocates tensor
// memory triggers only after its allocation (and the block-wide barrier behind it): a later kernel's CTA on the same
// SM can then never hold columns that this one still needs.  A dependent grid starts only when every CTA of its
// predecessor has triggered, hence is resident, so the resident CTAs are always a contiguous window of the chain
// and nobody waits on a CTA that cannot be scheduled.  (2) Nothing ahead of the wait reads memory that a kernel of
// the library writes (weights, LayerNorm gains: constant), except hints whose staleness costs time only.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

bool pdl_enabled();   // SDD_PDL != 0 (default on)

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// the same with a thread-block cluster of `cluster_x` consecutive CTAs along x (at most 8)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    unsigned cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster_x;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// tanh-GELU with the hardware tanh approximation (relative error about 2^-11): used where the result is
// rounded to bf16 (8 significant bits) anyway
__device__ __forceinline__ float gelu_tanh_fast(float x) {
  const float c = 0.7978845608028654f;
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(c * (x + 0.044715f * x * x * x)));
  return 0.5f * x * (1.f + t);
}

// device status word values (first error wins)
enum : int { DEV_OK = 0, DEV_TIMEOUT = 1, DEV_BAD_INDEX = 2 /* a commit past the token buffer */,
             DEV_BAD_TOKEN = 3 /* a token id outside the vocabulary */ };

}  // namespace sdd
