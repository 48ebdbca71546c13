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

// Programmatic dependent launch inside one call of the library. The FIRST kernel a public entry
// point launches is an ordinary launch: it starts once everything enqueued on the stream before
// the call has completed and its writes are visible, so every input of the call (activations,
// the KV cache and its lengths, index arrays written by an earlier call such as the escalation
// list, pruned-tree node counts or committed lengths) may be read by any kernel of the call at
// any time. Every LATER kernel of the same call is launched as a programmatic dependent of the
// kernel before it: its CTAs may be scheduled as soon as all CTAs of that kernel have called
// pdl_launch_dependents() (they do so at their start) and resources are free, so launch latency,
// prologues and tails inside a call overlap. Such a kernel calls pdl_wait() before its first read
// of anything an earlier kernel OF THE SAME CALL writes and before its first global write; the
// wait returns once all earlier kernels on the stream have completed and their writes are
// visible. Because every kernel waits before it completes, completion stays in stream order.
//
// EntryScope marks the extent of one public call on the calling thread (nested entry points,
// e.g. the fused pass calling the four steps, share the outermost scope).
struct EntryScope {
  EntryScope();
  ~EntryScope();
  EntryScope(const EntryScope&) = delete;
  EntryScope& operator=(const EntryScope&) = delete;
};
// True if a kernel was already launched inside the current outermost scope (the next launch may
// then be a programmatic dependent); records that a launch happens now.
bool entry_scope_next_launch_is_dependent();
// The next launch inside the current scope is an ordinary one again (after work was moved to or joined from
// another stream, where "the kernel before it" is not the kernel enqueued last).
void entry_scope_next_launch_ordinary();
// SMs the single-sequence LM head leaves free on its next launch from this thread (0 = none); consumed by
// that launch. The fused pass sets it when a small attention runs beside the LM head on a second stream.
void lm_reserve_sms_once(int n);

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                                    cudaStream_t st, unsigned cluster_x, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(block, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (entry_scope_next_launch_is_dependent()) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// CTAs the attention launch for these arguments will use (0 if the arguments are not accepted)
int attn_planned_ctas(const trispec_attn_args* a);

#define TRISPEC_CUDA_OK(expr)                        \
  do {                                               \
    cudaError_t _e = (expr);                         \
    if (_e != cudaSuccess) return TRISPEC_ERR_CUDA;  \
  } while (0)

}  // namespace trispec
