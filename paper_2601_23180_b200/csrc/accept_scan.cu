// Acceptance scan: greedy acceptance (Eq. 6), acceptance length tau_a (Eq. 7), margin
// predicate (Eq. 8), trusted prefix tau_m (Eq. 9) and the routing cases (i)/(ii)
// (Algorithm 1), evaluated along the path the greedy matches select in the draft tree.
// One warp per sequence. Each lane loads nodes `lane` and `lane + 32` of every per-node
// array once, coalesced (parent, token, top-1 index, the two probabilities); the margin test
// of all nodes becomes two ballots, and the walk then runs on registers: the current node's
// top-1 comes from a warp shuffle, the child match is a warp ballot. The accepted path is
// collected in registers and stored as one row. The ordered list of escalated sequence ids is
// made by the same block when the batch has at most 32 sequences, by further kernels otherwise.
#include "host_common.h"

namespace trispec {

constexpr int kScanThreads = 256;  // 8 sequences per block

// the proxy feature the routing criterion looks at (margin of Eq. 8 by default)
template <int kCrit>
__device__ __forceinline__ float scan_feature(const trispec_scan_args& a, long long idx) {
  if (kCrit == TRISPEC_CRIT_TOP1) return __ldg(a.in.p_top1 + idx);
  if (kCrit == TRISPEC_CRIT_ENTROPY) return __ldg(a.in.entropy + idx);
  return __ldg(a.in.p_top1 + idx) - __ldg(a.in.p_top2 + idx);
}

// The walk of one sequence by one warp; writes the sequence's outputs and returns its escalation flag.
// The routing criterion and the acceptance rule are compile-time switches: the kernel is short and
// latency-bound, and the plain case (margin rule, greedy acceptance) pays for nothing else.
// kAccept: TRISPEC_ACCEPT_GREEDY (arg-max match), _STOCHASTIC (Eq. 6 at temperature 1) or
// _TOKEN_SPECIFIC (the token-specific deferral rule of the SpecCascade baselines).
template <int kCrit, int kAccept>
__device__ __forceinline__ int scan_sequence(const trispec_scan_args& a, const long long b, const int lane) {
  const int T = a.T;
  const long long base = b * T;
  int32_t* path = a.path + base;
  const bool has0 = lane < T, has1 = lane + 32 < T;

  if (a.active && a.active[b] == 0) {
    if (has0) path[lane] = -1;
    if (has1) path[lane + 32] = -1;
    if (lane == 0) {
      a.accept_len[b] = 0;
      a.escalate[b] = 0;
      a.bonus_tok[b] = -1;
      a.last_node[b] = -1;
      if (a.near_thr) a.near_thr[b] = 0;
      if (a.esc_index) a.esc_index[b] = -1;
    }
    return 0;
  }

  // nodes `lane` and `lane + 32` of this sequence
  const bool proxy = (a.mode == TRISPEC_MODE_PROXY);
  int par0 = -2, par1 = -2, tok0 = 0, tok1 = 0, top0 = -1, top1v = -1;
  bool tr0 = true, tr1 = true, nr0 = false, nr1 = false;   // margin >= lambda / within 1e-3 of it
  constexpr bool stochastic = (kAccept == TRISPEC_ACCEPT_STOCHASTIC);
  constexpr bool token_rule = (kAccept == TRISPEC_ACCEPT_TOKEN_SPECIFIC);
  // token-specific rule: top-1 probability of this lane's nodes (the bar a child has to reach is
  // (1 - alpha) times its parent's) and the probability of the nodes' own drafted tokens
  float pt0 = 0.f, pt1 = 0.f, pd0 = -1.f, pd1 = -1.f;
  if (token_rule) {
    if (has0) { pt0 = __ldg(a.in.p_top1 + base + lane); if (lane > 0) pd0 = __ldg(a.in.p_draft + base + lane); }
    if (has1) { pt1 = __ldg(a.in.p_top1 + base + lane + 32); pd1 = __ldg(a.in.p_draft + base + lane + 32); }
  }
  if (has0) {
    par0 = __ldg(a.parent + base + lane); tok0 = __ldg(a.tok + base + lane);
    top0 = __ldg(a.in.top1_idx + base + lane);
    if (proxy) {
      const float f = scan_feature<kCrit>(a, base + lane);
      tr0 = (kCrit == TRISPEC_CRIT_ENTROPY) ? (f <= a.lambda) : (f >= a.lambda);
      nr0 = fabsf(f - a.lambda) < 1e-3f;
    }
  }
  if (has1) {
    par1 = __ldg(a.parent + base + lane + 32); tok1 = __ldg(a.tok + base + lane + 32);
    top1v = __ldg(a.in.top1_idx + base + lane + 32);
    if (proxy) {
      const float f = scan_feature<kCrit>(a, base + lane + 32);
      tr1 = (kCrit == TRISPEC_CRIT_ENTROPY) ? (f <= a.lambda) : (f >= a.lambda);
      nr1 = fabsf(f - a.lambda) < 1e-3f;
    }
  }
  // the margin test (Eq. 8) and the near-threshold mark of this lane's two nodes as four bits; the walk
  // fetches them from the current node's lane together with its top-1 (cur is the same in every lane, so
  // each lane picks its low or high node BEFORE the shuffle: one shuffle per value and step)
  const int flags = (tr0 ? 1 : 0) | (tr1 ? 2 : 0) | (nr0 ? 4 : 0) | (nr1 ? 8 : 0);
  // Bernoulli acceptance of Eq. 6 for every node at once: bit c = child c passes its test
  unsigned long long passes = ~0ull;
  if (stochastic) {
    bool ps0 = false, ps1 = false;
    if (has0 && lane > 0) {
      const float q = __ldg(a.q_draft + base + lane), pd = __ldg(a.in.p_draft + base + lane);
      ps0 = __ldg(a.u_accept + base + lane) < ((q > 0.f) ? fminf(1.f, pd / q) : 1.f);
    }
    if (has1) {
      const float q = __ldg(a.q_draft + base + lane + 32), pd = __ldg(a.in.p_draft + base + lane + 32);
      ps1 = __ldg(a.u_accept + base + lane + 32) < ((q > 0.f) ? fminf(1.f, pd / q) : 1.f);
    }
    passes = __ballot_sync(0xffffffffu, ps0) | (static_cast<unsigned long long>(__ballot_sync(0xffffffffu, ps1)) << 32);
  }
  // the compaction kernel only writes the leading entries of esc_index
  if (a.esc_index && lane == 0) a.esc_index[b] = -1;

  int cur = a.start_node ? a.start_node[b] : 0;
  if (cur < 0 || cur >= T) cur = 0;
  int n = 0, esc = 0, bonus = -1, near = 0;
  int path0 = -1, path1 = -1;   // entries `lane` and `lane + 32` of the accepted path
  // each accepted node has a larger index than the previous one: at most T iterations
  for (int it = 0; it < T; ++it) {
    const int src = cur & 31;
    const bool hi = cur >= 32;
    const int top1 = __shfl_sync(0xffffffffu, hi ? top1v : top0, src);
    if (proxy) {
      const int fl = __shfl_sync(0xffffffffu, flags, src) >> (hi ? 1 : 0);
      near += (fl >> 2) & 1;
      if (!(fl & 1)) { esc = 1; break; }
    }
    // greedy: the child whose token is the arg-max; stochastic: the first child that passed its
    // Bernoulli test; token-specific: the first child at least (1 - alpha) as probable as the arg-max
    unsigned m0, m1;
    if (token_rule) {
      const float bar = (1.f - a.alpha) * __shfl_sync(0xffffffffu, hi ? pt1 : pt0, src);
      m0 = __ballot_sync(0xffffffffu, par0 == cur && pd0 >= bar);
      m1 = __ballot_sync(0xffffffffu, par1 == cur && pd1 >= bar);
    } else {
      m0 = __ballot_sync(0xffffffffu, par0 == cur && (stochastic || tok0 == top1));
      m1 = __ballot_sync(0xffffffffu, par1 == cur && (stochastic || tok1 == top1));
    }
    if (stochastic) { m0 &= static_cast<unsigned>(passes); m1 &= static_cast<unsigned>(passes >> 32); }
    int nxt = -1;
    if (m0) nxt = __ffs(m0) - 1;
    else if (m1) nxt = 32 + __ffs(m1) - 1;
    if (nxt < 0) { bonus = stochastic ? -2 : top1; break; }
    if (lane == n) path0 = nxt;
    if (lane + 32 == n) path1 = nxt;
    ++n;
    cur = nxt;
  }
  if (has0) path[lane] = path0;
  if (has1) path[lane + 32] = path1;
  if (lane == 0) {
    a.accept_len[b] = n;
    a.escalate[b] = static_cast<uint8_t>(esc);
    a.bonus_tok[b] = bonus;
    a.last_node[b] = cur;
    if (a.near_thr) a.near_thr[b] = near;
  }
  return esc;
}

template <int kCrit, int kAccept>
__global__ void __launch_bounds__(kScanThreads)
accept_scan_kernel(trispec_scan_args a) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long b = static_cast<long long>(blockIdx.x) * (kScanThreads / 32) + (threadIdx.x >> 5);
  if (b >= a.B) return;
  scan_sequence<kCrit, kAccept>(a, b, lane);
}

// Up to 32 sequences (a decode batch): one block, one warp per sequence, and the ordered list of
// escalated sequences is made by the same block from a ballot of the flags, which saves the second
// launch of the general path.
constexpr int kScanSmallMax = 32;
template <int kCrit, int kAccept>
__global__ void __launch_bounds__(32 * kScanSmallMax)
accept_scan_small_kernel(trispec_scan_args a) {
  __shared__ int s_esc[kScanSmallMax];
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int esc = (warp < a.B) ? scan_sequence<kCrit, kAccept>(a, warp, lane) : 0;
  if (lane == 0) s_esc[warp] = esc;
  __syncthreads();
  if (warp == 0 && a.esc_index) {
    const bool flag = lane < a.B && lane < static_cast<int>(blockDim.x >> 5) && s_esc[lane] != 0;
    const unsigned m = __ballot_sync(0xffffffffu, flag);
    const int n = __popc(m);
    if (flag) a.esc_index[__popc(m & ((1u << lane) - 1u))] = lane;
    if (lane >= n && lane < a.B) a.esc_index[lane] = -1;
    if (lane == 0) *a.n_escalated = n;
  }
}

// Ordered compaction of the escalated sequence ids. A block owns 65536 consecutive flags; inside it a
// warp owns 2048 of them: lane l reads the 4-byte words l, l + 32, ... (coalesced), the block orders
// the warp totals with one barrier, and each word column is scattered with a warp scan, so that a warp
// writes consecutive entries of esc_index. Entries past the last escalated sequence were set to -1 by
// the scan kernel. Batches of more than 65536 sequences take one block per 65536 flags in two
// launches: the first leaves every block's count in a scratch array, the second starts each block at
// the sum of the counts before it (a caller without scratch gets one block that walks all rounds).
constexpr int kCompactThreads = 1024;
constexpr int kCompactWords = 16;                       // 4-byte words per lane and round
constexpr int kCompactPerWarp = 32 * kCompactWords * 4;  // flags per warp and round
constexpr long long kCompactPerBlock = static_cast<long long>(kCompactThreads / 32) * kCompactPerWarp;   // 65536

// flags of this warp's region as one bit per byte (0x01 per non-zero flag), and their count
__device__ __forceinline__ int compact_load(const uint8_t* __restrict__ escalate, long long B, long long region,
                                            bool word_ok, int lane, uint32_t (&w)[kCompactWords]) {
  if (word_ok && region + kCompactPerWarp <= B) {
    // whole region in range: sixteen independent coalesced loads in flight
#pragma unroll
    for (int j = 0; j < kCompactWords; ++j)
      w[j] = __ldg(reinterpret_cast<const uint32_t*>(escalate + region) + j * 32 + lane);
  } else {
#pragma unroll
    for (int j = 0; j < kCompactWords; ++j) {
      const long long first = region + (j * 32 + lane) * 4;
      uint32_t x = 0;
      for (int k = 0; k < 4; ++k)
        if (first + k < B) x |= static_cast<uint32_t>(escalate[first + k]) << (8 * k);
      w[j] = x;
    }
  }
  int cnt = 0;
#pragma unroll
  for (int j = 0; j < kCompactWords; ++j) {
    w[j] = __vcmpne4(w[j], 0u) & 0x01010101u;        // one bit per non-zero flag byte
    cnt += __popc(w[j]);
  }
  return cnt;
}

// first launch of the two-launch form: block_count[blk] = escalated sequences among the block's flags
__global__ void __launch_bounds__(kCompactThreads)
esc_count_kernel(const uint8_t* __restrict__ escalate, int B, int32_t* __restrict__ block_count) {
  __shared__ int warp_total[32];
  pdl_launch_dependents();
  pdl_wait();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool word_ok = (reinterpret_cast<uintptr_t>(escalate) & 3u) == 0;
  const long long region = blockIdx.x * kCompactPerBlock + static_cast<long long>(warp) * kCompactPerWarp;
  uint32_t w[kCompactWords];
  int cnt = compact_load(escalate, B, region, word_ok, lane, w);
  for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  if (lane == 0) warp_total[warp] = cnt;
  __syncthreads();
  if (warp == 0) {
    int t = warp_total[lane];
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) block_count[blockIdx.x] = t;
  }
}

// One block per 65536 flags when block_count is given (gridDim.x blocks, each starting at the sum of
// the counts of the blocks before it), else a single block that walks all rounds itself.
__global__ void __launch_bounds__(kCompactThreads)
esc_compact_kernel(const uint8_t* __restrict__ escalate, int B, int32_t* __restrict__ esc_index,
                   int32_t* __restrict__ n_escalated, const int32_t* __restrict__ block_count) {
  __shared__ int warp_total[2][32];
  __shared__ int s_start;
  pdl_launch_dependents();
  pdl_wait();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const bool word_ok = (reinterpret_cast<uintptr_t>(escalate) & 3u) == 0;
  int running = 0;      // escalated sequences before the current round (same value in every thread)
  long long start = 0, end = B;
  if (block_count) {
    // sum of the counts of the earlier blocks
    int part = 0;
    for (int j = tid; j < static_cast<int>(blockIdx.x); j += kCompactThreads) part += __ldg(block_count + j);
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) warp_total[0][warp] = part;
    __syncthreads();
    if (warp == 0) {
      int t = warp_total[0][lane];
      for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
      if (lane == 0) s_start = t;
    }
    __syncthreads();
    running = s_start;
    start = blockIdx.x * kCompactPerBlock;
    end = min(static_cast<long long>(B), start + kCompactPerBlock);
    __syncthreads();                                   // warp_total is reused below
  }
  int round = 0;
  for (; start < end; start += kCompactPerBlock, ++round) {
    const long long region = start + static_cast<long long>(warp) * kCompactPerWarp;
    uint32_t w[kCompactWords];
    int cnt = compact_load(escalate, B, region, word_ok, lane, w);
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);   // warp total
    if (lane == 0) warp_total[round & 1][warp] = cnt;
    __syncthreads();
    // every warp scans the 32 warp totals itself
    const int wt = warp_total[round & 1][lane];
    int wincl = wt;
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, wincl, o);
      if (lane >= o) wincl += v;
    }
    int off = running + __shfl_sync(0xffffffffu, wincl - wt, warp);
    running += __shfl_sync(0xffffffffu, wincl, 31);
    if (cnt) {
#pragma unroll
      for (int j = 0; j < kCompactWords; ++j) {
        const int c = __popc(w[j]);
        int incl = c;
        for (int o = 1; o < 32; o <<= 1) {
          const int v = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += v;
        }
        int dst = off + incl - c;
        uint32_t x = w[j];
        while (x) {
          const int bit = __ffs(x) - 1;
          x &= x - 1;
          esc_index[dst++] = static_cast<int32_t>(region + (j * 32 + lane) * 4 + (bit >> 3));
        }
        off += __shfl_sync(0xffffffffu, incl, 31);
      }
    }
  }
  // entries past the last escalated sequence already hold -1 (written by the scan kernel)
  if (tid == 0 && (!block_count || blockIdx.x == gridDim.x - 1)) *n_escalated = running;
}

}  // namespace trispec

extern "C" int trispec_accept_scan(const trispec_scan_args* a, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  if (!a || a->B <= 0 || a->T <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->T > 64) return TRISPEC_ERR_UNSUPPORTED;
  if (!a->parent || !a->tok || !a->in.top1_idx || !a->accept_len || !a->bonus_tok || !a->path || !a->last_node ||
      !a->escalate)
    return TRISPEC_ERR_INVALID_ARG;
  if (a->mode != TRISPEC_MODE_PROXY && a->mode != TRISPEC_MODE_TARGET) return TRISPEC_ERR_INVALID_ARG;
  if (a->criterion < TRISPEC_CRIT_MARGIN || a->criterion > TRISPEC_CRIT_ENTROPY) return TRISPEC_ERR_INVALID_ARG;
  if (a->mode == TRISPEC_MODE_PROXY) {
    if (a->criterion == TRISPEC_CRIT_MARGIN && (!a->in.p_top1 || !a->in.p_top2)) return TRISPEC_ERR_INVALID_ARG;
    if (a->criterion == TRISPEC_CRIT_TOP1 && !a->in.p_top1) return TRISPEC_ERR_INVALID_ARG;
    if (a->criterion == TRISPEC_CRIT_ENTROPY && !a->in.entropy) return TRISPEC_ERR_INVALID_ARG;
  }
  if ((a->n_escalated == nullptr) != (a->esc_index == nullptr)) return TRISPEC_ERR_INVALID_ARG;
  if ((a->q_draft == nullptr) != (a->u_accept == nullptr)) return TRISPEC_ERR_INVALID_ARG;
  // acceptance rule: the Bernoulli inputs select Eq. 6 when the rule field is left at its default
  int rule = a->accept_rule;
  if (rule == TRISPEC_ACCEPT_GREEDY && a->q_draft) rule = TRISPEC_ACCEPT_STOCHASTIC;
  if (rule < TRISPEC_ACCEPT_GREEDY || rule > TRISPEC_ACCEPT_TOKEN_SPECIFIC) return TRISPEC_ERR_INVALID_ARG;
  if (rule == TRISPEC_ACCEPT_STOCHASTIC && (!a->q_draft || !a->in.p_draft)) return TRISPEC_ERR_INVALID_ARG;
  if (rule == TRISPEC_ACCEPT_TOKEN_SPECIFIC &&
      (!a->in.p_draft || !a->in.p_top1 || !(a->alpha >= 0.f && a->alpha <= 1.f)))
    return TRISPEC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // kernel instance for (criterion, acceptance rule); TARGET mode reads no feature: margin instance
  const int crit = (a->mode == TRISPEC_MODE_PROXY) ? a->criterion : TRISPEC_CRIT_MARGIN;
  const int which = crit * 3 + rule;
  typedef void (*ScanKernel)(trispec_scan_args);
#define TRISPEC_SCAN_ROW(K, C) K<C, TRISPEC_ACCEPT_GREEDY>, K<C, TRISPEC_ACCEPT_STOCHASTIC>, K<C, TRISPEC_ACCEPT_TOKEN_SPECIFIC>
  static const ScanKernel small_k[9] = {TRISPEC_SCAN_ROW(accept_scan_small_kernel, TRISPEC_CRIT_MARGIN),
                                        TRISPEC_SCAN_ROW(accept_scan_small_kernel, TRISPEC_CRIT_TOP1),
                                        TRISPEC_SCAN_ROW(accept_scan_small_kernel, TRISPEC_CRIT_ENTROPY)};
  static const ScanKernel big_k[9] = {TRISPEC_SCAN_ROW(accept_scan_kernel, TRISPEC_CRIT_MARGIN),
                                      TRISPEC_SCAN_ROW(accept_scan_kernel, TRISPEC_CRIT_TOP1),
                                      TRISPEC_SCAN_ROW(accept_scan_kernel, TRISPEC_CRIT_ENTROPY)};
#undef TRISPEC_SCAN_ROW
  if (a->B <= kScanSmallMax) {
    TRISPEC_CUDA_OK(launch_dependent(small_k[which], 1u, static_cast<unsigned>(32 * a->B), 0, st, 1, *a));
    count_launch();
    return TRISPEC_OK;
  }
  const int per_block = kScanThreads / 32;
  unsigned grid = static_cast<unsigned>((static_cast<long long>(a->B) + per_block - 1) / per_block);
  TRISPEC_CUDA_OK(launch_dependent(big_k[which], grid, kScanThreads, 0, st, 1, *a));
  count_launch();
  if (a->esc_index) {
    const unsigned n_blk = static_cast<unsigned>((static_cast<long long>(a->B) + kCompactPerBlock - 1) / kCompactPerBlock);
    if (a->compact_scratch && n_blk > 1) {
      TRISPEC_CUDA_OK(launch_dependent(esc_count_kernel, n_blk, kCompactThreads, 0, st, 1,
                                       static_cast<const uint8_t*>(a->escalate), a->B, a->compact_scratch));
      count_launch();
      TRISPEC_CUDA_OK(launch_dependent(esc_compact_kernel, n_blk, kCompactThreads, 0, st, 1,
                                       static_cast<const uint8_t*>(a->escalate), a->B, a->esc_index, a->n_escalated,
                                       static_cast<const int32_t*>(a->compact_scratch)));
      count_launch();
    } else {
      TRISPEC_CUDA_OK(launch_dependent(esc_compact_kernel, 1, kCompactThreads, 0, st, 1,
                                       static_cast<const uint8_t*>(a->escalate), a->B, a->esc_index, a->n_escalated,
                                       static_cast<const int32_t*>(nullptr)));
      count_launch();
    }
  }
  return TRISPEC_OK;
}
