// Host-side helpers shared by the entry points: status codes, launch accounting, tensor-map
// encoding through the driver entry point (no link-time dependency on libcuda).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/trispec.h"

namespace trispec {

void count_launch(int n = 1);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Encodes a bf16 tiled tensor map with 128-byte swizzle. dims/box are innermost-first;
// strides_bytes has rank-1 entries (stride of dims 1..rank-1). Returns false on failure.
bool encode_tmap_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box);

// Same, through a small per-thread cache keyed by (base, rank, dims, strides, box): repeated
// calls with the same buffers (the steady state of a decode loop) skip the driver call.
bool cached_tmap_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box);

int device_sm_count();

// Raises the dynamic shared memory limit of `func` once per device.
int ensure_smem_limit(const void* func, int bytes, bool* done_per_device /* [64] */);

#define TRISPEC_CUDA_OK(expr)                        \
  do {                                               \
    cudaError_t _e = (expr);                         \
    if (_e != cudaSuccess) return TRISPEC_ERR_CUDA;  \
  } while (0)

}  // namespace trispec
