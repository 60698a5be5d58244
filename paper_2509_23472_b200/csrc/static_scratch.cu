// loract_weight_grad_static: the weight gradient from the factors for callers that cannot allocate.
//
// Some callers of this library are not allowed to obtain device memory at the point where they need the
// gradient: code running inside a framework's backward hook whose allocator is locked or already
// exhausted, a runtime that fixed its memory plan ahead of time, a process that must not touch
// cudaMalloc because another component owns the device's memory budget.  loract_weight_grad needs a
// caller-provided workspace for its intermediate T = U^T G; this variant needs none.  Its scratch is a
// fixed array inside the library image (below), so every GPU that loads the library holds
// kStaticScratchBytes of device memory until the process exits, and the problem size is limited.
#include <atomic>

#include "common.cuh"

namespace loract {
namespace {

constexpr size_t kStaticScratchBytes = 1u << 20;  // 1 MiB: status word + partial sums of T + T
constexpr size_t kStaticHeaderBytes = 256;

// Device code could name this array directly.  Host code cannot use the symbol as an address: on the
// host the name is only a stand-in, and a kernel handed `&g_static_scratch` from host code would fault
// or read the wrong memory.  The host asks the runtime for the array's device address (below).
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
// One slot per device, written once.  Two host threads that make their first call at the same moment both
// look the address up and store the same value, which is harmless; the atomic keeps the store and the loads
// well defined.  (A cudaDeviceReset in the same process invalidates the slot: callers that reset a device
// must not use this entry point afterwards.)
std::atomic<unsigned char*> g_scratch_addr[kMaxDevices];

// Set-up, once per device, with that device current: resolve the device address of the array.
cudaError_t static_scratch_address(unsigned char** out) {
  int dev = 0;
  LORACT_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  unsigned char* p = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!p) {
    LORACT_CUDA_TRY(cudaGetSymbolAddress((void**)&p, g_static_scratch));
    g_scratch_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return cudaSuccess;
}

}  // namespace
}  // namespace loract

using namespace loract;

extern "C" loract_status_t loract_weight_grad_static(const loract_desc_t* desc, const void* U, const void* V,
                                                     const void* G, int32_t g, int64_t ldg, float* dW,
                                                     int accumulate, void* stream) {
  const loract_status_t ds = check_desc(desc);   // the same descriptor rules as loract_weight_grad
  if (ds != LORACT_OK) return ds;
  if (!U || !V || !G || !dW) return LORACT_ERR_INVALID_ARG;
  if (g < 1 || g > 256 || ldg < g) return LORACT_ERR_INVALID_ARG;
  if (ldg % (desc->dtype == LORACT_BF16 ? 8 : 4)) return LORACT_ERR_ALIGNMENT;
  if (((uintptr_t)U & 15) || ((uintptr_t)V & 15) || ((uintptr_t)G & 15)) return LORACT_ERR_ALIGNMENT;
  const int r = desc->rank;
  // the fixed scratch must hold T and at least one partial sum of T
  const size_t t_bytes = ((size_t)r * g * 4 + 255) / 256 * 256;
  if (kStaticHeaderBytes + 2 * t_bytes > kStaticScratchBytes) return LORACT_ERR_UNSUPPORTED;  // rank * g too large
  unsigned char* base = nullptr;
  if (static_scratch_address(&base) != cudaSuccess) return LORACT_ERR_CUDA;
  const bool bf16 = desc->dtype == LORACT_BF16;
  int splits = bf16 ? gemm_tc_pick_splits(r, g, (int)desc->n_tokens, true, true) : (desc->n_tokens >= 4096 ? 16 : 1);
  const int max_splits = (int)((kStaticScratchBytes - kStaticHeaderBytes - t_bytes) / t_bytes);
  if (splits > max_splits) splits = max_splits;
  uint32_t* status = (uint32_t*)base;
  float* T = (float*)(base + kStaticHeaderBytes);
  float* partials = (float*)(base + kStaticHeaderBytes + t_bytes);
  cudaStream_t st = (cudaStream_t)stream;
  const int el = bf16 ? ELEM_BF16 : ELEM_F32;
  // the array keeps whatever the previous call left: clear the status word; T and the partial sums are
  // fully overwritten before they are read
  cudaError_t e = cudaMemsetAsync(status, 0, 4, st);
  GemmDesc t;  // T = U^T G, split over tokens
  t.M = r; t.N = g; t.K = (int)desc->n_tokens; t.a_mn = true; t.b_mn = true; t.lda = r; t.ldb = ldg;
  t.a_type = t.b_type = el;
  t.terms[0] = {U, G};
  t.out = OUT_F32; t.C0 = partials; t.ldc = g; t.splits = splits; t.split_stride = (int64_t)(t_bytes / 4);
  if (e == cudaSuccess) e = gemm_tc_supported(t) ? gemm_tc_launch(t, status, st) : gemm_simt_launch(t, st);
  if (e == cudaSuccess) e = reduce_partials_launch(partials, splits, t.split_stride, (int64_t)r * g, T, nullptr, st);
  if (e == cudaSuccess) {
    GemmDesc q;  // dW = V^T T
    q.M = (int)desc->d; q.N = g; q.K = r; q.a_mn = true; q.b_mn = true; q.lda = desc->d; q.ldb = g;
    q.a_type = el; q.b_type = ELEM_F32;
    q.terms[0] = {V, T};
    q.out = OUT_F32; q.C0 = dW; q.ldc = g; q.accumulate = accumulate != 0;
    e = gemm_simt_launch(q, st);
  }
  return e == cudaSuccess ? LORACT_OK : LORACT_ERR_CUDA;
}

// The status word of the static entry point lives in the library's own array, out of reach of
// loract_read_device_status; this reader copies it to the host.  Allocates nothing; synchronises `stream`.
extern "C" loract_status_t loract_weight_grad_static_status(uint32_t* out_host, void* stream) {
  if (!out_host) return LORACT_ERR_INVALID_ARG;
  unsigned char* base = nullptr;
  if (static_scratch_address(&base) != cudaSuccess) return LORACT_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(out_host, base, 4, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  return e == cudaSuccess ? LORACT_OK : LORACT_ERR_CUDA;
}
