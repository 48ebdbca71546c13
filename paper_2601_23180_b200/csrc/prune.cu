// Token pruning (routing case (ii) of "Adaptive Verification Routing"; ablation on token
// pruning): after the proxy accepted a prefix, only the subtree below the last accepted node
// goes to the target. One warp per sequence: each lane holds nodes `lane` and `lane + 32`.
// Membership is bit root of the node's ancestor mask; a ballot turns it into a 64-bit keep set,
// a node's new index is the number of kept nodes before it (popcount), and its new mask is its
// old mask restricted to kept nodes with the bits packed the same way. Integer work:
// 16 B in and 24 B out per node.
#include "host_common.h"

namespace trispec {

constexpr int kPruneThreads = 256;  // 8 sequences per block

// number of kept nodes with index < i
__device__ __forceinline__ int prune_rank(unsigned long long keep, int i) {
  return __popcll(keep & ((1ull << i) - 1ull));   // i < 64
}

// old ancestor mask -> mask over the new indices (only kept ancestors: those at or below the root)
__device__ __forceinline__ unsigned long long prune_pack_mask(unsigned long long old_mask, unsigned long long keep) {
  unsigned long long m = old_mask & keep, out = 0;
  while (m) {                       // at most depth + 1 bits
    const int j = __ffsll(static_cast<long long>(m)) - 1;
    m &= m - 1;
    out |= 1ull << prune_rank(keep, j);
  }
  return out;
}

__global__ void __launch_bounds__(kPruneThreads)
prune_tree_kernel(trispec_prune_args a) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long b = static_cast<long long>(blockIdx.x) * (kPruneThreads / 32) + (threadIdx.x >> 5);
  if (b >= a.B) return;
  const int T = a.T;
  const long long base = b * T;
  const bool has0 = lane < T, has1 = lane + 32 < T;
  const int r = __ldg(a.root + b);
  const bool skip = r < 0 || r >= T;

  int par0 = -1, par1 = -1, tok0 = -1, tok1 = -1;
  unsigned long long m0 = 0, m1 = 0;
  if (!skip && has0) { par0 = __ldg(a.parent + base + lane); tok0 = __ldg(a.tok + base + lane); m0 = __ldg(a.mask + base + lane); }
  if (!skip && has1) { par1 = __ldg(a.parent + base + lane + 32); tok1 = __ldg(a.tok + base + lane + 32); m1 = __ldg(a.mask + base + lane + 32); }
  const bool k0 = !skip && has0 && ((m0 >> r) & 1ull), k1 = !skip && has1 && ((m1 >> r) & 1ull);
  const unsigned long long keep =
      __ballot_sync(0xffffffffu, k0) | (static_cast<unsigned long long>(__ballot_sync(0xffffffffu, k1)) << 32);
  const int n_keep = __popcll(keep);

  // defaults for the entries beyond n_keep: every lane clears its two slots first if they are
  // past the end, the kept nodes then land in [0, n_keep)
  if (has0 && lane >= n_keep) {
    a.node_map[base + lane] = -1; a.parent_out[base + lane] = -1; a.tok_out[base + lane] = -1;
    if (a.mask_out) a.mask_out[base + lane] = 0ull;
    if (a.depth_out) a.depth_out[base + lane] = -1;
  }
  if (has1 && lane + 32 >= n_keep) {
    a.node_map[base + lane + 32] = -1; a.parent_out[base + lane + 32] = -1; a.tok_out[base + lane + 32] = -1;
    if (a.mask_out) a.mask_out[base + lane + 32] = 0ull;
    if (a.depth_out) a.depth_out[base + lane + 32] = -1;
  }
  if (k0) {
    const int j = prune_rank(keep, lane);
    const unsigned long long nm = prune_pack_mask(m0, keep);
    a.node_map[base + j] = lane;
    a.tok_out[base + j] = tok0;
    a.parent_out[base + j] = (lane == r) ? -1 : prune_rank(keep, par0);
    if (a.mask_out) a.mask_out[base + j] = nm;
    if (a.depth_out) a.depth_out[base + j] = __popcll(nm) - 1;
  }
  if (k1) {
    const int i = lane + 32;
    const int j = prune_rank(keep, i);
    const unsigned long long nm = prune_pack_mask(m1, keep);
    a.node_map[base + j] = i;
    a.tok_out[base + j] = tok1;
    a.parent_out[base + j] = (i == r) ? -1 : prune_rank(keep, par1);
    if (a.mask_out) a.mask_out[base + j] = nm;
    if (a.depth_out) a.depth_out[base + j] = __popcll(nm) - 1;
  }
  if (lane == 0) a.n_keep[b] = n_keep;
}

}  // namespace trispec

extern "C" int trispec_prune_tree(const trispec_prune_args* a, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  if (!a || a->B <= 0 || a->T <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->T > 64) return TRISPEC_ERR_UNSUPPORTED;
  if (!a->parent || !a->tok || !a->mask || !a->root || !a->n_keep || !a->node_map || !a->parent_out || !a->tok_out)
    return TRISPEC_ERR_INVALID_ARG;
  if (a->parent_out == a->parent || a->tok_out == a->tok || a->mask_out == a->mask) return TRISPEC_ERR_INVALID_ARG;
  const int per_block = kPruneThreads / 32;
  const unsigned grid = static_cast<unsigned>((static_cast<long long>(a->B) + per_block - 1) / per_block);
  TRISPEC_CUDA_OK(launch_dependent(prune_tree_kernel, grid, kPruneThreads, 0, static_cast<cudaStream_t>(stream), 1, *a));
  count_launch();
  return TRISPEC_OK;
}
