// KV commit of the accepted path (X <- X + Y of Algorithm 1 as the KV cache sees it): the keys
// and values of tree node 0 (the last committed token) and of the accepted draft nodes are
// appended to each sequence's cache. One block per sequence walks its appended rows (a row is
// Hkv x 128 bf16 for K and the same for V) with 16-byte loads and stores, four per thread in
// flight. A second, tiny kernel then writes the new lengths (so that they may be updated in place).
#include "host_common.h"

namespace trispec {

constexpr int kCommitThreads = 256;

struct CommitParams {
  int B, T, Hkv, paged, Lmax, num_blocks, max_blocks_per_seq;
  const uint4 *k_tree, *v_tree;     // [B][T][Hkv * 16] in 16-byte units
  uint4 *k_cache, *v_cache;
  const int32_t *block_table, *ctx_len, *path, *accept_len;
  const uint8_t* active;
  int32_t *ctx_len_out, *dev_status;
};

// rows the sequence appends (root + accepted nodes), or 0 if it is inactive / does not fit
__device__ __forceinline__ int commit_rows(const CommitParams& p, int b, int L) {
  if (p.active && p.active[b] == 0) return 0;
  int n = __ldg(p.accept_len + b);
  if (n < 0 || n >= p.T) n = 0;
  const int rows = n + 1;
  bool fits;
  if (!p.paged) {
    fits = L >= 0 && L + rows <= p.Lmax;
  } else {
    // every 64-token block the new rows fall into must be a valid entry of the table
    fits = L >= 0;
    const int first_blk = L / 64, last_blk = (L + rows - 1) / 64;
    for (int q = first_blk; fits && q <= last_blk; ++q) {
      if (q >= p.max_blocks_per_seq) { fits = false; break; }
      const int v = __ldg(p.block_table + static_cast<long long>(b) * p.max_blocks_per_seq + q);
      if (v < 0 || v >= p.num_blocks) fits = false;
    }
  }
  return fits ? rows : -1;
}

__global__ void __launch_bounds__(kCommitThreads)
kv_commit_kernel(const CommitParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const int L = __ldg(p.ctx_len + b);
  const int rows = commit_rows(p, b, L);
  if (rows < 0) {
    if (threadIdx.x == 0 && p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_NO_ROOM);   // sequence skipped
    return;
  }
  const int row16 = p.Hkv * 16;                  // 16-byte units per row (Hkv x 128 bf16)
  const int per_row = 2 * row16;                 // K then V
  const int total = rows * per_row;
  // four 16-byte units per thread and round, loads first: keeps 64 bytes per thread in flight
  for (int i0 = threadIdx.x; i0 < total; i0 += 4 * kCommitThreads) {
    uint4 val[4];
    long long dsti[4];
    bool isv[4], ok[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + u * kCommitThreads;
      ok[u] = i < total;
      dsti[u] = 0; isv[u] = false; val[u] = make_uint4(0, 0, 0, 0);
      if (!ok[u]) continue;
      const int j = i / per_row, e = i % per_row;
      int node = 0;
      if (j > 0) {
        node = __ldg(p.path + static_cast<long long>(b) * p.T + (j - 1));
        if (node < 0 || node >= p.T) { ok[u] = false; continue; }   // malformed path entry: nothing copied
      }
      const int t = L + j;
      isv[u] = e >= row16;
      const int off = isv[u] ? e - row16 : e;
      const long long src = (static_cast<long long>(b) * p.T + node) * row16 + off;
      if (!p.paged) {
        dsti[u] = (static_cast<long long>(b) * p.Lmax + t) * row16 + off;
      } else {
        const int blk = __ldg(p.block_table + static_cast<long long>(b) * p.max_blocks_per_seq + t / 64);
        dsti[u] = (static_cast<long long>(blk) * 64 + (t % 64)) * row16 + off;
      }
      val[u] = __ldg((isv[u] ? p.v_tree : p.k_tree) + src);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (ok[u]) (isv[u] ? p.v_cache : p.k_cache)[dsti[u]] = val[u];
  }
}

__global__ void __launch_bounds__(256)
kv_commit_len_kernel(const CommitParams p) {
  pdl_launch_dependents();
  pdl_wait();                                    // every copy block has read the old lengths
  const int b = blockIdx.x * 256 + threadIdx.x;
  if (b >= p.B) return;
  const int L = p.ctx_len[b];
  const int rows = commit_rows(p, b, L);
  p.ctx_len_out[b] = L + (rows > 0 ? rows : 0);
}

}  // namespace trispec

extern "C" int trispec_commit_kv(const trispec_commit_args* a, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  if (!a || a->B <= 0 || a->T <= 0 || a->Hkv <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->D != 128 || a->T > 64) return TRISPEC_ERR_UNSUPPORTED;
  if (!a->k_tree || !a->v_tree || !a->k_cache || !a->v_cache || !a->ctx_len || !a->path || !a->accept_len ||
      !a->ctx_len_out)
    return TRISPEC_ERR_INVALID_ARG;
  if (!aligned16(a->k_tree) || !aligned16(a->v_tree) || !aligned16(a->k_cache) || !aligned16(a->v_cache))
    return TRISPEC_ERR_INVALID_ARG;
  CommitParams p;
  p.B = a->B; p.T = a->T; p.Hkv = a->Hkv;
  if (a->kv_layout == TRISPEC_KV_CONTIGUOUS) {
    if (a->Lmax <= 0) return TRISPEC_ERR_INVALID_ARG;
    p.paged = 0;
  } else if (a->kv_layout == TRISPEC_KV_PAGED) {
    if (a->block_size != 64) return TRISPEC_ERR_UNSUPPORTED;
    if (!a->block_table || a->max_blocks_per_seq <= 0 || a->num_blocks <= 0) return TRISPEC_ERR_INVALID_ARG;
    p.paged = 1;
  } else {
    return TRISPEC_ERR_INVALID_ARG;
  }
  if (static_cast<long long>(a->B) * a->T > 0x7fffffffLL) return TRISPEC_ERR_UNSUPPORTED;
  p.Lmax = a->Lmax; p.num_blocks = a->num_blocks; p.max_blocks_per_seq = a->max_blocks_per_seq;
  p.k_tree = static_cast<const uint4*>(a->k_tree); p.v_tree = static_cast<const uint4*>(a->v_tree);
  p.k_cache = static_cast<uint4*>(a->k_cache); p.v_cache = static_cast<uint4*>(a->v_cache);
  p.block_table = a->block_table; p.ctx_len = a->ctx_len; p.path = a->path; p.accept_len = a->accept_len;
  p.active = a->active; p.ctx_len_out = a->ctx_len_out; p.dev_status = a->dev_status;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  TRISPEC_CUDA_OK(launch_dependent(kv_commit_kernel, static_cast<unsigned>(a->B), kCommitThreads, 0, st, 1, p));
  count_launch();
  TRISPEC_CUDA_OK(launch_dependent(kv_commit_len_kernel, static_cast<unsigned>((a->B + 255) / 256), 256, 0, st, 1, p));
  count_launch();
  return TRISPEC_OK;
}
