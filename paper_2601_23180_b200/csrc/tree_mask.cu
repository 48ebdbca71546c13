// Tree attention mask of a draft tree (Figure 4; tree configuration of Section 4.1): a node
// sees its ancestors and itself. One thread per node walks to the root; a block covers
// several sequences. Integer work, bytes are negligible (12 B in, 12 B out per node).
#include "host_common.h"

namespace trispec {

constexpr int kMaskThreads = 256;

__global__ void __launch_bounds__(kMaskThreads)
tree_mask_kernel(const int32_t* __restrict__ parent, uint64_t* __restrict__ mask, int32_t* __restrict__ depth,
                 long long n_nodes, int T) {
  pdl_launch_dependents();
  pdl_wait();
  long long idx = static_cast<long long>(blockIdx.x) * kMaskThreads + threadIdx.x;
  if (idx >= n_nodes) return;
  long long seq_base = (idx / T) * T;
  int i = static_cast<int>(idx - seq_base);
  const int32_t* par = parent + seq_base;
  uint64_t bits = 0;
  int steps = 0;
  int p = i;
  bool bad = false;
  // at most T hops: parent[p] < p is enforced on every hop, so the walk strictly descends
  while (p >= 0) {
    bits |= (1ull << p);
    ++steps;
    int np = __ldg(par + p);
    if (np >= p || np < -1 || (p == 0 && np != -1)) { bad = true; break; }
    p = np;
  }
  if (bad) { bits = 0; steps = 0; }
  mask[idx] = bits;
  if (depth) depth[idx] = steps - 1;
}

}  // namespace trispec

extern "C" int trispec_build_tree_mask(const trispec_tree_args* a, void* stream) {
  using namespace trispec;
  if (!a || !a->parent || !a->mask || a->B <= 0 || a->T <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->T > 64) return TRISPEC_ERR_UNSUPPORTED;
  long long n = static_cast<long long>(a->B) * a->T;
  unsigned grid = static_cast<unsigned>((n + kMaskThreads - 1) / kMaskThreads);
  TRISPEC_CUDA_OK(launch_dependent(tree_mask_kernel, grid, kMaskThreads, 0, static_cast<cudaStream_t>(stream), 1,
                                   a->parent, a->mask, a->depth, n, a->T));
  count_launch();
  return TRISPEC_OK;
}
