// erase_gemm_static: the GEMM entry point for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the moment they need a GEMM: code that
// runs inside a memory pool it does not own (an inference server or training framework that has
// handed all device memory to its own allocator), code under a real-time budget where an
// allocation's implicit device synchronisation is not acceptable, and code that may be asked to
// run while another component forbids allocation.  For them the split-K workspace and the
// status word live in a fixed array in the library's own device image instead.
#include <cuda_runtime.h>

#include <atomic>
#include <string>

#include "../../include/erase.h"
#include "gemm_tc.cuh"
#include "kernels.cuh"

using namespace erase;

namespace {

// Scratch shared by every call on a device: [0, ERASE_STATIC_WS_FLOATS) split-K partial sums,
// then one status word and two tile-scheduler words.  Held by every device that loads the library until the process exits.
constexpr size_t kWsFloats = ERASE_STATIC_WS_FLOATS;
static __device__ __align__(256) float g_static_scratch[kWsFloats + 64];

constexpr int kMaxDevices = 64;
std::atomic<float*> g_scratch_addr[kMaxDevices];  // device address of g_static_scratch, per device (host threads may race to fill it: same value)

thread_local std::string g_static_error;

}  // namespace

extern "C" {

ERASE_API const char* erase_gemm_static_error(void) { return g_static_error.c_str(); }

ERASE_API erase_status erase_gemm_static(int32_t dtype, int32_t M, int32_t N, int32_t K, const void* A, int64_t sa_m,
                                         int64_t sa_k, const void* B, int64_t sb_n, int64_t sb_k, void* C, int64_t ldc,
                                         int32_t c_f32, int32_t splits, int32_t engine, void* stream) {
  auto fail = [&](erase_status st, const std::string& msg) {
    g_static_error = "erase_gemm_static: " + msg;
    return st;
  };
  if ((dtype != ERASE_F32 && dtype != ERASE_BF16) || M < 1 || N < 1 || K < 1 || !A || !B || !C || splits < 1 ||
      (engine != 0 && engine != 1) || ldc < N || (sa_m != 1 && sa_k != 1) || (sb_n != 1 && sb_k != 1))
    return fail(ERASE_EINVAL, "bad argument");
  const bool bf = dtype == ERASE_BF16;
  const int out_f32 = (c_f32 || !bf) ? 1 : 0;
  if (splits > 1 && !out_f32) return fail(ERASE_EINVAL, "split-K needs a float result (c_f32)");
  const size_t need = splits > 1 ? (size_t)splits * (size_t)M * (size_t)N : 0;
  if (need > kWsFloats)
    return fail(ERASE_EINVAL, "split-K workspace of " + std::to_string(need) + " floats exceeds the static maximum of " +
                                  std::to_string(kWsFloats) + " (splits*M*N must not exceed ERASE_STATIC_WS_FLOATS)");

  // One-time set-up per device: the array's name is only a host-side handle; kernels need its
  // device address, which cudaGetSymbolAddress returns for the device that is current.
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(ERASE_ECUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(ERASE_EUNSUPPORTED, "device ordinal out of range");
  if (!g_scratch_addr[dev].load(std::memory_order_acquire)) {
    float* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) {
      cudaGetLastError();
      return fail(ERASE_ECUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
    }
    g_scratch_addr[dev].store(ptr, std::memory_order_release);
  }
  float* ws = g_scratch_addr[dev].load(std::memory_order_acquire);
  int* status = reinterpret_cast<int*>(ws + kWsFloats);

  cudaStream_t st = (cudaStream_t)stream;
  GemmArgs g;
  g.M = M; g.N = N; g.K = K;
  g.A = A; g.sa_m = sa_m; g.sa_k = sa_k;
  g.B = B; g.sb_n = sb_n; g.sb_k = sb_k;
  g.C = C; g.ldc = ldc; g.c_f32 = out_f32;
  g.splits = splits;
  g.ws = splits > 1 ? ws : nullptr;
  g.epi.ld_aux = N;
  if (engine == 1 && (!bf || !tc_gemm_supported(g)))
    return fail(ERASE_EUNSUPPORTED, "the tensor-core kernel does not take this shape/alignment/dtype");

  // The array keeps the previous call's contents.  The partial sums need no clearing (every
  // element that is read was written by this call); the status word must start at zero.
  e = cudaMemsetAsync(status, 0, 4 * sizeof(int), st);   // status word and the two tile-scheduler words after it
  if (e != cudaSuccess) return fail(ERASE_ECUDA, std::string("status clear: ") + cudaGetErrorString(e));
  if (engine == 1) {
    TcPlan plan;
    if (!tc_gemm_plan(g, status, &plan)) return fail(ERASE_EUNSUPPORTED, "TMA descriptor encoding failed");
    plan.sched = status + 1;
    e = tc_gemm_launch(g, plan, st);
  } else {
    e = gemm_simt(g, bf, st);
  }
  if (e != cudaSuccess) return fail(ERASE_ECUDA, std::string("launch: ") + cudaGetErrorString(e));
  if (splits > 1) {
    e = splitk_reduce(ws, splits, (long long)M * N, N, (float*)C, ldc, st);
    if (e != cudaSuccess) return fail(ERASE_ECUDA, std::string("reduce launch: ") + cudaGetErrorString(e));
  }
  int hst = 0;
  e = cudaMemcpyAsync(&hst, status, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(ERASE_ECUDA, std::string("execution: ") + cudaGetErrorString(e));
  if (hst != 0) return fail(ERASE_ETIMEOUT, "a bounded device-side wait expired (code " + std::to_string(hst) + ")");
  g_static_error.clear();
  return ERASE_OK;
}

}  // extern "C"
