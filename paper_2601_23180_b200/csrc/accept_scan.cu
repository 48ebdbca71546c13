// Acceptance scan: greedy acceptance (Eq. 6), acceptance length tau_a (Eq. 7), margin
// predicate (Eq. 8), trusted prefix tau_m (Eq. 9) and the routing cases (i)/(ii)
// (Algorithm 1), evaluated along the path the greedy matches select in the draft tree.
// One warp per sequence: each lane keeps two tree nodes in registers, the child match is a
// warp ballot. A second single-block kernel compacts the escalated sequence ids in order.
#include "host_common.h"

namespace trispec {

constexpr int kScanThreads = 256;  // 8 sequences per block

__global__ void __launch_bounds__(kScanThreads)
accept_scan_kernel(trispec_scan_args a) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long b = static_cast<long long>(blockIdx.x) * (kScanThreads / 32) + (threadIdx.x >> 5);
  if (b >= a.B) return;
  const int T = a.T;
  const long long base = b * T;
  int32_t* path = a.path + base;

  if (a.active && a.active[b] == 0) {
    if (lane < T) path[lane] = -1;
    if (lane + 32 < T) path[lane + 32] = -1;
    if (lane == 0) {
      a.accept_len[b] = 0;
      a.escalate[b] = 0;
      a.bonus_tok[b] = -1;
      a.last_node[b] = -1;
      if (a.near_thr) a.near_thr[b] = 0;
    }
    return;
  }

  // nodes `lane` and `lane + 32` of this sequence
  int par0 = -2, par1 = -2, tok0 = 0, tok1 = 0;
  if (lane < T) { par0 = __ldg(a.parent + base + lane); tok0 = __ldg(a.tok + base + lane); }
  if (lane + 32 < T) { par1 = __ldg(a.parent + base + lane + 32); tok1 = __ldg(a.tok + base + lane + 32); }

  int cur = a.start_node ? a.start_node[b] : 0;
  if (cur < 0 || cur >= T) cur = 0;
  int n = 0, esc = 0, bonus = -1, near = 0;
  // each accepted node has a larger index than the previous one: at most T iterations
  for (int it = 0; it < T; ++it) {
    const int top1 = __ldg(a.in.top1_idx + base + cur);
    if (a.mode == TRISPEC_MODE_PROXY) {
      const float margin = __ldg(a.in.p_top1 + base + cur) - __ldg(a.in.p_top2 + base + cur);
      if (fabsf(margin - a.lambda) < 1e-3f) ++near;
      if (!(margin >= a.lambda)) { esc = 1; break; }
    }
    const unsigned m0 = __ballot_sync(0xffffffffu, par0 == cur && tok0 == top1);
    const unsigned m1 = __ballot_sync(0xffffffffu, par1 == cur && tok1 == top1);
    int nxt = -1;
    if (m0) nxt = __ffs(m0) - 1;
    else if (m1) nxt = 32 + __ffs(m1) - 1;
    if (nxt < 0) { bonus = top1; break; }
    if (lane == 0) path[n] = nxt;
    ++n;
    cur = nxt;
  }
  if (lane >= n && lane < T) path[lane] = -1;
  if (lane + 32 >= n && lane + 32 < T) path[lane + 32] = -1;
  if (lane == 0) {
    a.accept_len[b] = n;
    a.escalate[b] = static_cast<uint8_t>(esc);
    a.bonus_tok[b] = bonus;
    a.last_node[b] = cur;
    if (a.near_thr) a.near_thr[b] = near;
  }
}

// Ordered compaction of the escalated sequence ids: one block, 16 flags per thread per round.
constexpr int kCompactThreads = 1024;
__global__ void __launch_bounds__(kCompactThreads)
esc_compact_kernel(const uint8_t* __restrict__ escalate, int B, int32_t* __restrict__ esc_index,
                   int32_t* __restrict__ n_escalated) {
  __shared__ int warp_excl[32];
  __shared__ int running;
  pdl_launch_dependents();
  pdl_wait();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) running = 0;
  __syncthreads();
  for (long long start = 0; start < B; start += static_cast<long long>(kCompactThreads) * 16) {
    const long long first = start + static_cast<long long>(tid) * 16;
    unsigned bits = 0;
    for (int j = 0; j < 16; ++j) {
      long long s = first + j;
      if (s < B && escalate[s]) bits |= (1u << j);
    }
    const int cnt = __popc(bits);
    int incl = cnt;  // inclusive prefix inside the warp
    for (int o = 1; o < 32; o <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_excl[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const int w = warp_excl[lane];
      int wi = w;
      for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += v;
      }
      warp_excl[lane] = wi - w;  // exclusive prefix of the warp totals
    }
    __syncthreads();
    const int off = running + warp_excl[warp] + (incl - cnt);
    int k = 0;
    for (int j = 0; j < 16; ++j)
      if (bits & (1u << j)) esc_index[off + (k++)] = static_cast<int32_t>(first + j);
    __syncthreads();                                   // everyone has read `running`
    if (tid == kCompactThreads - 1) running = off + cnt;  // last thread: total so far
    __syncthreads();
  }
  const int total = running;
  for (long long s = static_cast<long long>(total) + tid; s < B; s += kCompactThreads) esc_index[s] = -1;
  if (tid == 0) *n_escalated = total;
}

}  // namespace trispec

extern "C" int trispec_accept_scan(const trispec_scan_args* a, void* stream) {
  using namespace trispec;
  if (!a || a->B <= 0 || a->T <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->T > 64) return TRISPEC_ERR_UNSUPPORTED;
  if (!a->parent || !a->tok || !a->in.top1_idx || !a->accept_len || !a->bonus_tok || !a->path || !a->last_node ||
      !a->escalate)
    return TRISPEC_ERR_INVALID_ARG;
  if (a->mode != TRISPEC_MODE_PROXY && a->mode != TRISPEC_MODE_TARGET) return TRISPEC_ERR_INVALID_ARG;
  if (a->mode == TRISPEC_MODE_PROXY && (!a->in.p_top1 || !a->in.p_top2)) return TRISPEC_ERR_INVALID_ARG;
  if ((a->n_escalated == nullptr) != (a->esc_index == nullptr)) return TRISPEC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int per_block = kScanThreads / 32;
  unsigned grid = static_cast<unsigned>((static_cast<long long>(a->B) + per_block - 1) / per_block);
  TRISPEC_CUDA_OK(launch_dependent(accept_scan_kernel, grid, kScanThreads, 0, st, 1, *a));
  count_launch();
  if (a->esc_index) {
    TRISPEC_CUDA_OK(launch_dependent(esc_compact_kernel, 1, kCompactThreads, 0, st, 1,
                                     static_cast<const uint8_t*>(a->escalate), a->B, a->esc_index, a->n_escalated));
    count_launch();
  }
  return TRISPEC_OK;
}
