// An allocation-free variant of the copied-gradient step (FP8 GEMM into FP32 scratch, then copy-add into the
// destination).  Some callers cannot allocate device memory at the point where they need this operation -- a
// plugin running inside another framework's memory-pool lock, a callback on a thread that must not touch the
// allocator, an embedded runtime whose memory is fully partitioned at start-up -- so here the scratch is a fixed
// array that is part of the library image on every GPU that loads it.
#include <atomic>
#include <cstdint>

#include "error.h"
#include "kernels.h"
#include "qe.h"

using qe::fail;

namespace {

constexpr uint64_t kStagingElems = 1ull << 20;  // FP32 elements: 4 MiB, e.g. one 1024 x 1024 gradient slice

// Device-resident scratch.  In host code this name is only a handle for the runtime's symbol table, not an address a
// kernel could use; the usable address is looked up once per device below.
static __device__ __align__(256) float g_staging[kStagingElems];

constexpr int kMaxDevices = 16;
// One cached address per device.  Atomic, so that host threads making their first calls at the same time do not race
// on it (each would look up and store the same value).
std::atomic<float*> g_staging_addr[kMaxDevices];

// First use on a device (that device current): resolve the device address of g_staging.
int32_t staging_address(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(QE_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(QE_ERR_UNSUPPORTED, "device ordinal %d beyond %d", dev, kMaxDevices);
  float* p = g_staging_addr[dev].load(std::memory_order_acquire);
  if (!p) {
    e = cudaGetSymbolAddress((void**)&p, g_staging);
    if (e != cudaSuccess || !p) return fail(QE_ERR_CUDA, "cudaGetSymbolAddress(staging): %s", cudaGetErrorString(e));
    g_staging_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return QE_OK;
}

}  // namespace

extern "C" int32_t qe_gemm_fp8_staged_noalloc(const void* a, uint32_t a_fmt, const void* b, uint32_t b_fmt, uint32_t M,
                                              uint32_t Nn, uint32_t Kc, const float* alpha_a, const float* alpha_b,
                                              float* dst, int32_t accumulate, uint32_t* status_dev, void* stream) {
  if (!dst) return fail(QE_ERR_BAD_ARG, "dst_dev is null");
  if ((uintptr_t)dst & 15u) return fail(QE_ERR_BAD_ARG, "dst_dev must be 16-byte aligned");
  const uint64_t elems = (uint64_t)M * Nn;
  if (elems > kStagingElems)
    return fail(QE_ERR_UNSUPPORTED, "M*N = %llu exceeds the built-in staging area of %llu FP32 elements",
                (unsigned long long)elems, (unsigned long long)kStagingElems);
  float* staging = nullptr;
  int32_t st = staging_address(&staging);
  if (st != QE_OK) return st;
  // D = (A . B^T) * alpha written in full to the staging area (nothing in it needs clearing first) ...
  st = qe_gemm_fp8(a, a_fmt, b, b_fmt, M, Nn, Kc, alpha_a, alpha_b, staging, 1u, nullptr, status_dev, stream);
  if (st != QE_OK) return st;
  // ... then dst (=|+=) staging, the same copy-add kernel the copied-gradient path uses.
  return qe_accumulate(dst, staging, elems, accumulate, stream);
}

extern "C" uint64_t qe_noalloc_staging_elems(void) { return kStagingElems; }
