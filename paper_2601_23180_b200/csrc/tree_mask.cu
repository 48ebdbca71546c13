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
                 long long n_seq, int T, int32_t* __restrict__ status) {
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
    // not a tree (a parent out of range, or a second root): reported through the status word
    const bool bad = (has0 && (q0 == -2 || (lane != 0 && q0 == -1))) || (has1 && q1 < 0);
    if (__any_sync(0xffffffffu, bad) && lane == 0 && status) atomicExch(status, TRISPEC_ERR_BAD_TREE);
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

// Large batches (thousands of sequences): one THREAD per sequence. Parents precede children, so a
// node's mask is its parent's mask plus its own bit, and one pass over the nodes in order does it:
// about ten instructions per node for one thread, against a whole warp climbing level by level
// above (which is the better shape for a decode batch, where sequences are few). A block takes 64
// sequences: all 256 threads load their parents (16-byte loads) into shared memory, 64 threads walk,
// all 256 threads write masks and depths back, coalesced. The (sequence, node) pair of a flat element
// index is carried along incrementally (no division by the run-time T in the copy loops), and the
// masks sit in shared memory sequence-major with an odd pitch: the walkers (one sequence per lane)
// and the copy-out (consecutive elements per lane) both touch distinct banks.
constexpr int kMaskBlockSeqs = 64, kMaskBlockThreads = 256;
constexpr int kMaskParPitch = kMaskBlockSeqs + 1;   // bytes per node row of the parent table: a lane's four
                                                    // consecutive nodes, and its neighbours' (4 nodes on), hit distinct banks
constexpr int kMaskSeqPitch = 65;                   // masks per sequence row (T <= 64, odd)

// element index e = seq * T + node, advanced by `step` elements
struct MaskElem {
  int seq, node;
  __device__ __forceinline__ void advance(int dseq, int dnode, int T) {
    seq += dseq;
    node += dnode;
    if (node >= T) { node -= T; ++seq; }
  }
  __device__ __forceinline__ MaskElem next(int T) const {
    MaskElem r = *this;
    if (++r.node == T) { r.node = 0; ++r.seq; }
    return r;
  }
};

__global__ void __launch_bounds__(kMaskBlockThreads)
tree_mask_block_kernel(const int32_t* __restrict__ parent, uint64_t* __restrict__ mask, int32_t* __restrict__ depth,
                       long long n_seq, int T, int32_t* __restrict__ status) {
  __shared__ signed char sPar[64 * kMaskParPitch];
  __shared__ unsigned long long sMask[kMaskBlockSeqs * kMaskSeqPitch];
  pdl_launch_dependents();
  pdl_wait();
  const long long s0 = static_cast<long long>(blockIdx.x) * kMaskBlockSeqs;
  const int n_here = static_cast<int>(min(static_cast<long long>(kMaskBlockSeqs), n_seq - s0));
  const int n_elem = n_here * T;
  const int32_t* src = parent + s0 * T;
  // parents -> shared memory as bytes ([node][sequence]); anything outside [-1, 62] becomes -2
  auto put = [&](const MaskElem& e, int v) {
    sPar[e.node * kMaskParPitch + e.seq] = static_cast<signed char>((v >= -1 && v < 63) ? v : -2);
  };
  if ((n_elem & 3) == 0 && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    const int4* src4 = reinterpret_cast<const int4*>(src);
    const int first = 4 * threadIdx.x, step = 4 * kMaskBlockThreads;
    MaskElem e0 = {first / T, first % T};
    const int dseq = step / T, dnode = step % T;
#pragma unroll 2
    for (int q = threadIdx.x; q < (n_elem >> 2); q += kMaskBlockThreads) {
      const int4 v = __ldg(src4 + q);
      const MaskElem e1 = e0.next(T), e2 = e1.next(T), e3 = e2.next(T);
      put(e0, v.x); put(e1, v.y); put(e2, v.z); put(e3, v.w);
      e0.advance(dseq, dnode, T);
    }
  } else {
    MaskElem e0 = {static_cast<int>(threadIdx.x) / T, static_cast<int>(threadIdx.x) % T};
    const int dseq = kMaskBlockThreads / T, dnode = kMaskBlockThreads % T;
    for (int e = threadIdx.x; e < n_elem; e += kMaskBlockThreads) {
      put(e0, __ldg(src + e));
      e0.advance(dseq, dnode, T);
    }
  }
  __syncthreads();
  if (threadIdx.x < n_here) {
    const int t = threadIdx.x;
    unsigned long long* row = sMask + t * kMaskSeqPitch;
    bool bad = false;
    for (int i = 0; i < T; ++i) {
      const int par = sPar[i * kMaskParPitch + t];
      unsigned long long m;
      if (par == -1) {
        m = 1ull << i;                                      // a root
        bad |= (i != 0);                                    // a second root: not a tree
      } else if (par < 0 || par >= i) {
        m = 0ull;                                           // malformed: flagged, not followed
        bad = true;
      } else {
        const unsigned long long pm = row[par];
        m = pm ? (pm | (1ull << i)) : 0ull;                 // a malformed ancestor spoils the walk
      }
      row[i] = m;
    }
    if (bad && status) atomicExch(status, TRISPEC_ERR_BAD_TREE);
  }
  __syncthreads();
  uint64_t* dst = mask + s0 * T;
  int32_t* ddst = depth ? depth + s0 * T : nullptr;
  auto get = [&](const MaskElem& e) -> unsigned long long { return sMask[e.seq * kMaskSeqPitch + e.node]; };
  if ((n_elem & 1) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0 &&
      (!ddst || (reinterpret_cast<uintptr_t>(ddst) & 7u) == 0)) {
    const int first = 2 * threadIdx.x, step = 2 * kMaskBlockThreads;
    MaskElem e0 = {first / T, first % T};
    const int dseq = step / T, dnode = step % T;
#pragma unroll 2
    for (int q = threadIdx.x; q < (n_elem >> 1); q += kMaskBlockThreads) {   // two masks = 16 bytes per store
      const unsigned long long m0 = get(e0), m1 = get(e0.next(T));
      reinterpret_cast<ulonglong2*>(dst)[q] = make_ulonglong2(m0, m1);
      if (ddst) reinterpret_cast<int2*>(ddst)[q] = make_int2(__popcll(m0) - 1, __popcll(m1) - 1);
      e0.advance(dseq, dnode, T);
    }
  } else {
    MaskElem e0 = {static_cast<int>(threadIdx.x) / T, static_cast<int>(threadIdx.x) % T};
    const int dseq = kMaskBlockThreads / T, dnode = kMaskBlockThreads % T;
    for (int e = threadIdx.x; e < n_elem; e += kMaskBlockThreads) {
      const unsigned long long m = get(e0);
      dst[e] = m;
      if (ddst) ddst[e] = __popcll(m) - 1;
      e0.advance(dseq, dnode, T);
    }
  }
}

}  // namespace trispec

extern "C" int trispec_build_tree_mask(const trispec_tree_args* a, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  if (!a || !a->parent || !a->mask || a->B <= 0 || a->T <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->T > 64) return TRISPEC_ERR_UNSUPPORTED;
  const long long n = a->B;
  if (n >= 2048) {   // enough sequences to fill the chip with a thread each
    unsigned grid = static_cast<unsigned>((n + kMaskBlockSeqs - 1) / kMaskBlockSeqs);
    TRISPEC_CUDA_OK(launch_dependent(tree_mask_block_kernel, grid, kMaskBlockThreads, 0,
                                     static_cast<cudaStream_t>(stream), 1, a->parent, a->mask, a->depth, n, a->T,
                                     a->dev_status));
    count_launch();
    return TRISPEC_OK;
  }
  const int per_block = (kMaskThreads / 32) * kMaskSeqPerWarp;
  unsigned grid = static_cast<unsigned>((n + per_block - 1) / per_block);
  TRISPEC_CUDA_OK(launch_dependent(tree_mask_kernel, grid, kMaskThreads, 0, static_cast<cudaStream_t>(stream), 1,
                                   a->parent, a->mask, a->depth, n, a->T, a->dev_status));
  count_launch();
  return TRISPEC_OK;
}
