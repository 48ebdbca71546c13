#include <string.h>

#include <atomic>
#include <mutex>

#include "host_common.h"

namespace trispec {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

namespace {
thread_local int tl_scope_depth = 0;
thread_local bool tl_scope_launched = false;
}  // namespace
EntryScope::EntryScope() {
  if (tl_scope_depth++ == 0) tl_scope_launched = false;
}
EntryScope::~EntryScope() { --tl_scope_depth; }
void entry_scope_next_launch_ordinary() { tl_scope_launched = false; }
bool entry_scope_next_launch_is_dependent() {
  const bool dependent = tl_scope_depth > 0 && tl_scope_launched;
  tl_scope_launched = true;
  return dependent;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

bool encode_tmap_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[5], gstr[5];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
  }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), gdim, gstr, bx, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

namespace {
struct TmapKey {
  const void* base;
  int rank;
  uint64_t dims[4], strides[3];
  uint32_t box[4];
  int device;
};
struct TmapEntry {
  TmapKey key;
  CUtensorMap map;
  bool valid;
};
constexpr int kTmapCache = 32;
}  // namespace

bool cached_tmap_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims,
                      const uint64_t* strides_bytes, const uint32_t* box) {
  thread_local TmapEntry cache[kTmapCache] = {};
  thread_local int next = 0;
  TmapKey k;
  memset(&k, 0, sizeof(k));
  k.base = base;
  k.rank = rank;
  for (int i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) k.strides[i] = strides_bytes[i];
  if (cudaGetDevice(&k.device) != cudaSuccess) return false;
  for (int i = 0; i < kTmapCache; ++i)
    if (cache[i].valid && memcmp(&cache[i].key, &k, sizeof(k)) == 0) {
      *out = cache[i].map;
      return true;
    }
  if (!encode_tmap_bf16(out, base, rank, dims, strides_bytes, box)) return false;
  cache[next].key = k;
  cache[next].map = *out;
  cache[next].valid = true;
  next = (next + 1) % kTmapCache;
  return true;
}

int ensure_smem_limit(const void* func, int bytes, bool* done_per_device) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRISPEC_ERR_CUDA;
  if (dev >= 0 && dev < 64 && done_per_device[dev]) return TRISPEC_OK;
  if (cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
    return TRISPEC_ERR_CUDA;
  if (dev >= 0 && dev < 64) done_per_device[dev] = true;
  return TRISPEC_OK;
}

int device_sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace trispec

extern "C" const char* trispec_status_string(int s) {
  switch (s) {
    case TRISPEC_OK: return "ok";
    case TRISPEC_ERR_INVALID_ARG: return "invalid argument";
    case TRISPEC_ERR_UNSUPPORTED: return "unsupported shape";
    case TRISPEC_ERR_WORKSPACE: return "workspace too small";
    case TRISPEC_ERR_CUDA: return "CUDA call failed";
    case TRISPEC_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case TRISPEC_ERR_BAD_BLOCK: return "block table entry out of range (device status)";
    case TRISPEC_ERR_SMEM_ALIGN: return "shared-memory window misplaced (device status)";
    case TRISPEC_ERR_NO_ROOM: return "no room in the KV cache for the committed rows (device status)";
    case TRISPEC_ERR_BAD_LENGTH: return "context length out of range (device status)";
    case TRISPEC_ERR_BAD_TREE: return "parent array is not a tree (device status)";
    case TRISPEC_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

extern "C" long long trispec_launch_count(void) { return trispec::g_launches.load(std::memory_order_relaxed); }
