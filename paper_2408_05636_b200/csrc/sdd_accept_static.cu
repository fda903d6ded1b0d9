// sdd_accept_logits_static: the stand-alone acceptance step for callers that cannot allocate
// device memory.  Its scratch (the per-chunk soft-max statistics) lives in a fixed array in the
// library's device image instead of a caller-provided buffer.
#include <mutex>

#include "sdd_kernels.h"

namespace {

constexpr size_t kStaticScratchBytes = SDD_ACCEPT_STATIC_SCRATCH_BYTES;

// Every GPU that loads this library holds one copy of this array until the process exits.
static __device__ __align__(256) unsigned char g_accept_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};   // device address of g_accept_scratch, per device ordinal

// The array's name is only a host-side handle here; kernels need its device address, which the
// runtime reports per device.  Looked up once per device, with that device current.
int static_scratch(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SDD_E_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_accept_scratch);
    if (e != cudaSuccess || p == nullptr) return SDD_E_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return SDD_OK;
}

}  // namespace

extern "C" int32_t sdd_accept_logits_static(const float* logits_p, const float* logits_q, const int32_t* draft_ids,
                                            int32_t rows, int32_t gamma, int32_t V, float temp_p, float temp_q,
                                            uint64_t seed, uint64_t round, int32_t* n_accept, int32_t* out_ids,
                                            float* accept_prob, void* stream) {
  using namespace sdd;
  if (!logits_p || !logits_q || !draft_ids || !n_accept || !out_ids || !accept_prob) return SDD_E_ARG;
  if (rows < 1 || rows > 65535 || gamma < 1 || gamma > 256 || V < 2) return SDD_E_ARG;
  if (!(temp_p >= 0.f) || !(temp_q >= 0.f) || ((temp_p == 0.f) != (temp_q == 0.f))) return SDD_E_ARG;
  if (((uintptr_t)logits_p & 15u) || ((uintptr_t)logits_q & 15u)) return SDD_E_ARG;
  const int chunks = stats_chunks_for(V);
  const unsigned long long need = (unsigned long long)rows * (2ull * gamma + 1) * chunks * sizeof(float2);
  if (need > kStaticScratchBytes) return SDD_E_WORKSPACE;   // problem too large for the fixed scratch
  void* scratch = nullptr;
  const int s = static_scratch(&scratch);
  if (s != SDD_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  const float itp = temp_p > 0.f ? 1.f / temp_p : 0.f, itq = temp_q > 0.f ? 1.f / temp_q : 0.f;
  float2* partial = (float2*)scratch;
  const long long rows_p = (long long)rows * (gamma + 1), rows_q = (long long)rows * gamma;
  // every (row, chunk) pair that the second kernel reads is written by the first one in this same call,
  // so nothing in the shared array has to be cleared between calls
  if (launch_row_stats(logits_p, rows_p, logits_q, itp == 0.f ? 0 : rows_q, V, itp, itq, partial, st) != cudaSuccess)
    return SDD_E_CUDA;
  if (launch_accept(logits_p, logits_q, draft_ids, nullptr, nullptr, partial, chunks, partial + rows_p * chunks, chunks, rows, gamma, V, itp, itq,
                    make_key(seed), (uint32_t)round, nullptr, accept_prob, n_accept, nullptr, out_ids, st) != cudaSuccess)
    return SDD_E_CUDA;
  return SDD_OK;
}
