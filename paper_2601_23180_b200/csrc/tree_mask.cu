// Tree attention mask of a draft tree (Figure 4; tree configuration of Section 4.1): a node
// sees its ancestors and itself. One warp per sequence: each lane holds the parents of nodes
// `lane` and `lane + 32` (one coalesced load) and all nodes climb to the root together, one
// shuffle per level; a warp takes two sequences and issues their loads together. Integer
// work; 4 B in and 12 B out per node.
#include "host_common.h"

namespace trispec {

constexpr int kMaskThreads = 256;
constexpr int kMaskSeqPerWarp = 2;  // sequences per warp: their loads are issued together

__global__ void __launch_bounds__(kMaskThreads)
tree_mask_kernel(const int32_t* __restrict__ parent, uint64_t* __restrict__ mask, int32_t* __restrict__ depth,
                 long long n_seq, int T) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long w = static_cast<long long>(blockIdx.x) * (kMaskThreads / 32) + (threadIdx.x >> 5);
  const long long b0 = w * kMaskSeqPerWarp;
  if (b0 >= n_seq) return;
  const bool has0 = lane < T, has1 = lane + 32 < T;
  int par0[kMaskSeqPerWarp], par1[kMaskSeqPerWarp];
#pragma unroll
  for (int u = 0; u < kMaskSeqPerWarp; ++u) {
    const long long base = (b0 + u) * T;
    const bool live = b0 + u < n_seq;
    par0[u] = (live && has0) ? __ldg(parent + base + lane) : -1;
    par1[u] = (live && has1) ? __ldg(parent + base + lane + 32) : -1;
  }
#pragma unroll
  for (int u = 0; u < kMaskSeqPerWarp; ++u) {
    if (b0 + u >= n_seq) break;
    const long long base = (b0 + u) * T;
    // parent[i] must satisfy -1 <= parent[i] < i (and parent[0] == -1); anything else marks the
    // node, and every node whose walk meets it, as malformed: mask 0, depth -1
    int q0 = par0[u], q1 = par1[u];
    if (has0 && !(q0 >= -1 && q0 < lane && (lane != 0 || q0 == -1))) q0 = -2;
    if (has1 && !(q1 >= -1 && q1 < lane + 32)) q1 = -2;
    // both parents of a lane in one register (a byte each, biased by 2), so that a walk needs
    // one shuffle per level
    const int packed = (q0 + 2) | ((q1 + 2) << 8);
    uint64_t bits0 = 0, bits1 = 0;
    int p0 = has0 ? lane : -1, p1 = has1 ? lane + 32 : -1;   // node each walk currently stands on
    // the walks strictly descend, so T levels are enough; stop as soon as every walk has ended
    for (int it = 0; it < T; ++it) {
      if (!__any_sync(0xffffffffu, (p0 & p1) >= 0)) break;   // some walk is still on a node
      const int g0 = __shfl_sync(0xffffffffu, packed, p0 & 31);
      const int g1 = __shfl_sync(0xffffffffu, packed, p1 & 31);
      if (p0 >= 0) { bits0 |= (1ull << p0); p0 = ((g0 >> ((p0 >> 5) << 3)) & 0xff) - 2; }
      if (p1 >= 0) { bits1 |= (1ull << p1); p1 = ((g1 >> ((p1 >> 5) << 3)) & 0xff) - 2; }
    }
    // a walk ends at -1 (above the root) or at -2 (malformed parent on the way)
    if (p0 != -1) bits0 = 0;
    if (p1 != -1) bits1 = 0;
    if (has0) { mask[base + lane] = bits0; if (depth) depth[base + lane] = __popcll(bits0) - 1; }
    if (has1) { mask[base + lane + 32] = bits1; if (depth) depth[base + lane + 32] = __popcll(bits1) - 1; }
  }
}

}  // namespace trispec

extern "C" int trispec_build_tree_mask(const trispec_tree_args* a, void* stream) {
  using namespace trispec;
  if (!a || !a->parent || !a->mask || a->B <= 0 || a->T <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->T > 64) return TRISPEC_ERR_UNSUPPORTED;
  const long long n = a->B;
  const int per_block = (kMaskThreads / 32) * kMaskSeqPerWarp;
  unsigned grid = static_cast<unsigned>((n + per_block - 1) / per_block);
  TRISPEC_CUDA_OK(launch_dependent(tree_mask_kernel, grid, kMaskThreads, 0, static_cast<cudaStream_t>(stream), 1,
                                   a->parent, a->mask, a->depth, n, a->T));
  count_launch();
  return TRISPEC_OK;
}
