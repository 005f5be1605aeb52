// Column sums of dY (the bias gradient) for callers that must not allocate device memory.
//
// The regular path takes its scratch (one fp32 row of partial sums per slab of rows) from
// the caller's workspace, which somebody had to cudaMalloc.  Some callers cannot do that:
// an enqueue hook of an inference runtime that hands out a fixed arena and forbids further
// allocation, a latency-critical loop that must never enter the allocator, or a process
// whose device memory pool is owned by another component.  For them the scratch lives in
// this file as a fixed-size device array that is part of the library's device code.  The
// first call on a device resolves the array's address; under lazy module loading that is also
// the moment the runtime may load the device code, array included, so that call is a warm-up
// to be made before the region that must not allocate and before any stream capture.  Calls
// share the array: calls that may overlap on the GPU race.
#include <atomic>

#include "internal.h"

namespace {

// Largest N accepted: 64 slabs x 16384 columns x 4 bytes = 4 MiB, resident on every GPU
// that loads the library until the process exits.
constexpr int64_t NOALLOC_MAX_N = 16384;

static __device__ __align__(256) float g_colsum_scratch[efqat::COLSUM_SLABS * NOALLOC_MAX_N];

// Device address of g_colsum_scratch per CUDA device, resolved on first use (any thread may
// be the first; all of them resolve the same value).  In host code the symbol itself is only
// a stand-in; kernels must be given the resolved address.
std::atomic<float*> g_scratch_addr[64];

}  // namespace

extern "C" int efqat_colsum_noalloc(int dtype, const void* dY, int64_t M, int64_t N, float* db,
                                    efqat_stream_t stream) {
  if (!dY || !db) return EFQAT_ERR_NULL;
  if (dtype != EFQAT_F32 && dtype != EFQAT_BF16) return EFQAT_ERR_DTYPE;
  if (M < 1 || N < 1) return EFQAT_ERR_SHAPE;
  if (N > NOALLOC_MAX_N) return EFQAT_ERR_TOO_LARGE;
  if ((N & 7) || (reinterpret_cast<uintptr_t>(dY) & 15)) return EFQAT_ERR_ALIGN;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return EFQAT_ERR_CUDA;
  float* scratch = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    // once per device, with that device current
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&scratch), g_colsum_scratch) != cudaSuccess || !scratch)
      return EFQAT_ERR_CUDA;
    g_scratch_addr[dev].store(scratch, std::memory_order_release);
  }
  // Every scratch element the second stage reads is written by the first stage of the same
  // call, so nothing has to be cleared between calls.
  efqat::launch_colsum(dY, dtype, M, N, scratch, db, stream);
  return cudaGetLastError() == cudaSuccess ? EFQAT_OK : EFQAT_ERR_CUDA;
}
