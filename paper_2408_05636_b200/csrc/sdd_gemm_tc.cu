// bf16 tensor-core GEMM for sm_100a:  C[M, N] = A[M, K] * W[N, K]^T  (fp32 accumulate) with fused epilogues.
//
// One CTA computes one 128 x BN accumulator tile that lives in tensor memory (TMEM).  Operand tiles
// (128 x 64 and BN x 64 bf16, K-major, 128-byte swizzle) are brought into a shared-memory ring by TMA
// (cp.async.bulk.tensor, one elected producer thread), consumed by tcgen05.mma issued from one elected
// thread, and the finished accumulator is read back with tcgen05.ld by four epilogue warps.
//
// Orientation.  NORMAL: MMA-M axis = activation rows, MMA-N axis = output features (large-M GEMMs of
// the drafter).  SWAP: MMA-M axis = output features (rows of W), MMA-N axis = tokens -- for the target's
// verification forward, where only gamma+1 tokens exist and the kernel is a weight-streaming pass; the
// epilogue then writes the transposed tile so that consecutive lanes write consecutive features.
//
// Every wait on an mbarrier is bounded: when the limit passes the thread raises the CTA's abort flag and
// the device status word, all roles leave their loops, the producer waits (bounded) for the copies it
// still has in flight, TMEM is freed and the CTA returns.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <map>
#include <mutex>
#include <tuple>

#include "sdd_kernels.h"

namespace sdd {

namespace tc {

constexpr int BM = 128;          // MMA M
constexpr int BK = 64;           // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int STAGES = 4;
constexpr int THREADS = 192;     // warp 0: TMA producer, warp 1: MMA issuer + TMEM owner, warps 2-5: epilogue
constexpr long long WAIT_LIMIT_CYCLES = 2000000000ll;   // about one second

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait; false = gave up (abort flag raised by this or another thread)
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
      *abort_flag = 1;
      if (status != nullptr) atomicCAS(status, DEV_OK, DEV_TIMEOUT);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  // K-major, 128-byte swizzle: 8-row groups are 1024 bytes apart (SBO), LBO unused (1), descriptor version 1
  return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

template <int BN>
__host__ __device__ constexpr uint32_t make_idesc() {
  // D = fp32, A = B = bf16, both K-major, N = BN, M = 128
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <int BN>
constexpr int stage_bytes() { return BM * BK * 2 + BN * BK * 2; }
template <int BN>
constexpr int smem_bytes() { return STAGES * stage_bytes<BN>() + 1024 /*alignment slack*/ + 256 /*barriers*/; }

template <int BN, bool SWAP>
__global__ void __launch_bounds__(THREADS)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, int rows_a,
               int rows_b, int K, int epi, const float* __restrict__ bias, void* __restrict__ out, int ldc, int* status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = base + STAGES * stage_bytes<BN>();
  // barrier block: full[STAGES], empty[STAGES], tmem_full, then the TMEM base address and the abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t tmem_full_bar = bar_base + 8u * (2 * STAGES);
  uint8_t* generic_base = smem_raw + (base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(generic_base + STAGES * stage_bytes<BN>() + 8 * (2 * STAGES + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(generic_base + STAGES * stage_bytes<BN>() + 8 * (2 * STAGES + 1) + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * BM;      // offset along the A operand's rows (MMA M axis)
  const int n0 = blockIdx.x * BN;      // offset along the B operand's rows (MMA N axis)
  const int num_kb = (K + BK - 1) / BK;
  constexpr uint32_t TMEM_COLS = BN < 32 ? 32 : BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(tmem_full_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, status)) break;
        mbar_expect_tx(full_bar(s), (uint32_t)stage_bytes<BN>());
        const uint32_t sa = base + s * stage_bytes<BN>();
        tma_load_2d(sa, &map_a, full_bar(s), kb * BK, m0);
        tma_load_2d(sa + BM * BK * 2, &map_b, full_bar(s), kb * BK, n0);
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
        const uint32_t sa = base + s * stage_bytes<BN>();
        const uint64_t da = make_smem_desc(sa), db = make_smem_desc(sa + BM * BK * 2);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k)
          umma(tmem_base, da + (uint64_t)(k * UMMA_K * 2 / 16), db + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
               (kb > 0 || k > 0) ? 1u : 0u);
        umma_commit(empty_bar(s));     // frees the stage once these MMAs have read it
      }
      if (ok) umma_commit(tmem_full_bar);
    }
  } else {
    // epilogue warps 2..5 own TMEM lane quarters (warp id % 4)
    const int q = warp & 3;
    // every lane waits; the outcome is made warp-uniform because tcgen05.ld is a warp-wide instruction
    const bool ready = __all_sync(0xffffffffu, mbar_wait(tmem_full_bar, 0u, abort_flag, status));
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ready) {
      const int r = m0 + q * 32 + lane;          // index along the A operand's rows
      const bool r_ok = r < rows_a;
#pragma unroll 1
      for (int cc = 0; cc < BN / 32; ++cc) {
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(cc * 32), v);
        const int c0 = n0 + cc * 32;             // index along the B operand's rows
        if (!SWAP) {
          // out[r][c]: r = token row, c = feature
          if (r_ok) {
            if (epi == EPI_STORE || epi == EPI_GELU) {
              __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out) + (long long)r * ldc + c0;
              if (c0 + 32 <= rows_b && (ldc & 7) == 0) {
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                  uint32_t pk[4];
#pragma unroll
                  for (int e = 0; e < 4; ++e) {
                    float x0 = __uint_as_float(v[g * 8 + 2 * e]) + (bias ? bias[c0 + g * 8 + 2 * e] : 0.f);
                    float x1 = __uint_as_float(v[g * 8 + 2 * e + 1]) + (bias ? bias[c0 + g * 8 + 2 * e + 1] : 0.f);
                    if (epi == EPI_GELU) { x0 = gelu_tanh(x0); x1 = gelu_tanh(x1); }
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
                    pk[e] = *reinterpret_cast<uint32_t*>(&h2);
                  }
                  *reinterpret_cast<uint4*>(o + g * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
              } else {
                for (int j = 0; j < 32; ++j) {
                  if (c0 + j < rows_b) {
                    float x = __uint_as_float(v[j]) + (bias ? bias[c0 + j] : 0.f);
                    if (epi == EPI_GELU) x = gelu_tanh(x);
                    o[j] = __float2bfloat16_rn(x);
                  }
                }
              }
            } else {
              float* o = reinterpret_cast<float*>(out) + (long long)r * ldc + c0;
              for (int j = 0; j < 32; ++j) {
                if (c0 + j < rows_b) {
                  const float x = __uint_as_float(v[j]) + (bias ? bias[c0 + j] : 0.f);
                  if (epi == EPI_RESIDUAL) o[j] += x; else o[j] = x;
                }
              }
            }
          }
        } else {
          // out[c][r]: c = token, r = feature; consecutive lanes write consecutive features
          const float bv = (bias != nullptr && r_ok) ? bias[r] : 0.f;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int c = c0 + j;
            if (r_ok && c < rows_b) {
              float x = __uint_as_float(v[j]) + bv;
              const long long o = (long long)c * ldc + r;
              if (epi == EPI_STORE) reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(x);
              else if (epi == EPI_GELU) reinterpret_cast<__nv_bfloat16*>(out)[o] = __float2bfloat16_rn(gelu_tanh(x));
              else if (epi == EPI_RESIDUAL) reinterpret_cast<float*>(out)[o] += x;
              else reinterpret_cast<float*>(out)[o] = x;
            }
          }
        }
      }
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
// host side: tensor maps (cached per pointer / shape / box) and launch
// ---------------------------------------------------------------------------------------------
static PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
static std::mutex g_mu;
static std::map<std::tuple<const void*, long long, int, int>, CUtensorMap> g_maps;

static cudaError_t get_encode() {
  if (g_encode != nullptr) return cudaSuccess;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
  g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
  return cudaSuccess;
}

// 2-D bf16 tensor [rows, cols] with row stride ld elements; box = box_rows x 64 columns, 128-byte swizzle
static cudaError_t get_map(const void* ptr, long long rows, int cols, int ld, int box_rows, CUtensorMap* out) {
  std::lock_guard<std::mutex> lock(g_mu);
  cudaError_t e = get_encode();
  if (e != cudaSuccess) return e;
  // the leading dimension is part of the key through `cols` of the callers (all operands are dense: ld == cols)
  auto key = std::make_tuple(ptr, rows * 4096ll + box_rows, cols, ld);
  auto it = g_maps.find(key);
  if (it != g_maps.end()) { *out = it->second; return cudaSuccess; }
  if ((reinterpret_cast<uintptr_t>(ptr) & 15u) != 0 || (ld * 2) % 16 != 0) return cudaErrorInvalidValue;
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  if (g_maps.size() > 8192) g_maps.clear();
  g_maps[key] = m;
  *out = m;
  return cudaSuccess;
}

template <int BN, bool SWAP>
static cudaError_t launch_cfg(const CUtensorMap& ma, const CUtensorMap& mb, int rows_a, int rows_b, int K, int epi,
                              const float* bias, void* out, int ldc, int* status, cudaStream_t st) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, SWAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<BN>());
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  dim3 grid((rows_b + BN - 1) / BN, (rows_a + BM - 1) / BM);
  gemm_tc_kernel<BN, SWAP><<<grid, THREADS, smem_bytes<BN>(), st>>>(ma, mb, rows_a, rows_b, K, epi, bias, out, ldc, status);
  return cudaGetLastError();
}

}  // namespace tc

// A: activations [M rows used, capacity a_cap rows, K], W: weights [N, K]; both dense bf16.
cudaError_t launch_gemm_tc(const __nv_bfloat16* A, long long a_cap, const __nv_bfloat16* W, const float* bias, int M, int N,
                           int K, int epi, void* out, int ldc, int bn_hint, int* status, cudaStream_t st) {
  using namespace tc;
  if (M <= 0 || N <= 0) return cudaSuccess;
  CUtensorMap ma, mb;
  cudaError_t e;
  if (M <= 64) {
    // SWAP: A operand = weights (box 128 rows), B operand = tokens (box BN rows)
    const int bn = M <= 32 ? 32 : 64;
    if ((e = get_map(W, N, K, K, BM, &ma)) != cudaSuccess) return e;
    if ((e = get_map(A, a_cap, K, K, bn, &mb)) != cudaSuccess) return e;
    if (bn == 32) return launch_cfg<32, true>(ma, mb, N, M, K, epi, bias, out, ldc, status, st);
    return launch_cfg<64, true>(ma, mb, N, M, K, epi, bias, out, ldc, status, st);
  }
  int bn = bn_hint;
  if (bn != 32 && bn != 64 && bn != 128 && bn != 256) {
    const long long mt = (M + BM - 1) / BM;
    bn = 32;
    for (int cand : {256, 128, 64}) {
      if (mt * ((N + cand - 1) / cand) >= 120) { bn = cand; break; }
    }
  }
  if ((e = get_map(A, a_cap, K, K, BM, &ma)) != cudaSuccess) return e;
  if ((e = get_map(W, N, K, K, bn, &mb)) != cudaSuccess) return e;
  switch (bn) {
    case 256: return launch_cfg<256, false>(ma, mb, M, N, K, epi, bias, out, ldc, status, st);
    case 128: return launch_cfg<128, false>(ma, mb, M, N, K, epi, bias, out, ldc, status, st);
    case 64: return launch_cfg<64, false>(ma, mb, M, N, K, epi, bias, out, ldc, status, st);
    default: return launch_cfg<32, false>(ma, mb, M, N, K, epi, bias, out, ldc, status, st);
  }
}

}  // namespace sdd
