// Bonus sampling (Algorithm 1: x_bonus ~ p_{tau_a + 1}) by the Gumbel-max identity: one more
// pass over W in which every CTA adds counter-based Gumbel noise to the logits of its
// vocabulary range and keeps, per sequence, the largest perturbed logit. Three kernels:
//   sample_gather_kernel    copies row (b, last_node[b]) of h into a compact [B][d] buffer
//                           (zero row for sequences that need no sample)
//   sample_gemm_kernel      z = Hc W^T on tcgen05 (M tile = 128 sequences, N tile <= 256,
//                           K block 64, 4-stage TMA ring, fp32 accumulators double-buffered in
//                           TMEM); epilogue: y = scale * z + G(seed, step, b, v), running
//                           (max, argmax) per row in registers, one partial per (row, range).
//                           The pass is bound by streaming W from HBM; the MMAs and the Philox
//                           rounds of the few live rows hide under it.
//   sample_finalize_kernel  one warp per sequence merges the partials and writes the token.
#include <math.h>

#include "host_common.h"
#include "sm100.cuh"

namespace trispec {

constexpr int SM_BM = 128, SM_BN = 256, SM_BK = 64, SM_STAGES = 4;
constexpr int SM_A_BYTES = SM_BM * SM_BK * 2;   // 16 KB
constexpr int SM_B_BYTES = SM_BN * SM_BK * 2;   // 32 KB
constexpr int SM_BOX_BYTES = 64 * SM_BK * 2;
constexpr int SM_STAGE_BYTES = SM_A_BYTES + SM_B_BYTES;
constexpr int SM_THREADS = 192;
constexpr int SM_SMEM_BYTES = SM_STAGES * SM_STAGE_BYTES + 1024 + 256;

struct SamplePartial { float y; int idx; };

struct SampleParams {
  int B, T, d, V, n_mt, n_ranges;
  float scale;
  unsigned int seed_lo, seed_hi, step_lo, step_hi;
  const uint16_t* h;
  uint16_t* hc;              // [n_mt * 128][d] compact rows
  const int32_t* last_node;
  int32_t* bonus_tok;
  float* sample_value;
  SamplePartial* partial;    // [n_ranges][n_mt * 128]
  int32_t* dev_status;
};

// Philox-4x32 with 10 rounds (Salmon et al., SC'11), written from the published definition
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const unsigned int hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const unsigned int hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}
__device__ __forceinline__ float gumbel_from_word(unsigned int w) {
  const float u = (static_cast<float>(w >> 9) + 0.5f) * (1.0f / 8388608.0f);   // exact, inside (0, 1)
  return -logf(-logf(u));
}

__global__ void __launch_bounds__(256)
sample_gather_kernel(const SampleParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const bool live = b < p.B && __ldg(p.bonus_tok + b) == -2;
  int node = live ? __ldg(p.last_node + b) : 0;
  const bool ok = live && node >= 0 && node < p.T;
  const uint4* src = reinterpret_cast<const uint4*>(p.h + (static_cast<long long>(b) * p.T + (ok ? node : 0)) * p.d);
  uint4* dst = reinterpret_cast<uint4*>(p.hc + static_cast<long long>(b) * p.d);
  for (int i = threadIdx.x; i < p.d / 8; i += 256) dst[i] = ok ? __ldg(src + i) : make_uint4(0, 0, 0, 0);
}

// vocabulary range r of n_ranges in tiles of at most 256 columns (multiples of 16)
struct SampleTiles {
  int u0, units, n_tiles;
  __device__ SampleTiles(int V, int n_ranges, int r) {
    const int V16 = (V + 15) >> 4;
    u0 = static_cast<int>((static_cast<long long>(V16) * r) / n_ranges);
    units = static_cast<int>((static_cast<long long>(V16) * (r + 1)) / n_ranges) - u0;
    n_tiles = (units + 15) >> 4;
  }
  __device__ void tile(int t, int& n0, int& nw) const {
    const int a = (units * t) / n_tiles, b = (units * (t + 1)) / n_tiles;
    n0 = (u0 + a) << 4;
    nw = (b - a) << 4;
  }
};

__global__ void __launch_bounds__(SM_THREADS, 1)
sample_gemm_kernel(const __grid_constant__ CUtensorMap tmap_hc, const __grid_constant__ CUtensorMap tmap_w,
                   const SampleParams p) {
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base_u32 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base_u32 - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SM_STAGES * SM_STAGE_BYTES);
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = bars + SM_STAGES;
  uint64_t* tmem_full = bars + 2 * SM_STAGES;
  uint64_t* tmem_empty = bars + 2 * SM_STAGES + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * SM_STAGES + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int mt = blockIdx.x % p.n_mt;
  const int range = blockIdx.x / p.n_mt;
  const SampleTiles tiles(p.V, p.n_ranges, range);
  const int n_kb = p.d / SM_BK;

  if (threadIdx.x == 0) {
    for (int i = 0; i < SM_STAGES; ++i) { mbar_init(full_bar + i, 1); mbar_init(empty_bar + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tmem_full + i, 1); mbar_init(tmem_empty + i, 4); }
    fence_mbar_init();
  }
  if (warp == 5) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  if (warp == 4 && lane == 0) { prefetch_tmap(&tmap_hc); prefetch_tmap(&tmap_w); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();   // the compact rows come from the gather kernel

  if (warp == 4) {
    if (lane == 0) {   // ---------------------------------------------------------- TMA producer
      int stage = 0;
      uint32_t phase = 0;
      for (int t = 0; t < tiles.n_tiles; ++t) {
        int n0, nw;
        tiles.tile(t, n0, nw);
        const int nbox = (nw + 63) >> 6;
        const uint32_t tx = static_cast<uint32_t>(2 + nbox) * SM_BOX_BYTES;
        for (int kb = 0; kb < n_kb; ++kb) {
          mbar_wait(empty_bar + stage, phase ^ 1u, p.dev_status);
          uint8_t* sa = smem + stage * SM_STAGE_BYTES;
          uint8_t* sb = sa + SM_A_BYTES;
          mbar_expect_tx(full_bar + stage, tx);
          tma_load_2d(sa, &tmap_hc, full_bar + stage, kb * SM_BK, mt * SM_BM);
          tma_load_2d(sa + SM_BOX_BYTES, &tmap_hc, full_bar + stage, kb * SM_BK, mt * SM_BM + 64);
          for (int j = 0; j < nbox; ++j)
            tma_load_2d(sb + j * SM_BOX_BYTES, &tmap_w, full_bar + stage, kb * SM_BK, n0 + 64 * j);
          if (++stage == SM_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {   // ---------------------------------------------------------- MMA issuer
      int stage = 0;
      uint32_t phase = 0;
      for (int t = 0; t < tiles.n_tiles; ++t) {
        int n0, nw;
        tiles.tile(t, n0, nw);
        const int buf = t & 1;
        mbar_wait(tmem_empty + buf, ((t >> 1) & 1u) ^ 1u, p.dev_status);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * SM_BN);
        const uint32_t idesc = idesc_bf16(SM_BM, nw, false, false);
        for (int kb = 0; kb < n_kb; ++kb) {
          mbar_wait(full_bar + stage, phase, p.dev_status);
          tc_fence_after();
          const uint32_t sa = base_u32 + stage * SM_STAGE_BYTES;
          const uint64_t adesc = smem_desc_sw128(sa, 1024, 16);
          const uint64_t bdesc = smem_desc_sw128(sa + SM_A_BYTES, 1024, 16);
#pragma unroll
          for (int k = 0; k < SM_BK / 16; ++k) tc_mma_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | k) != 0);
          tc_commit(empty_bar + stage);
          if (++stage == SM_STAGES) { stage = 0; phase ^= 1u; }
        }
        tc_commit(tmem_full + buf);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3)
    const int row = warp * 32 + lane;             // TMEM lane = sequence slot of this M tile
    const int b = mt * SM_BM + row;
    const bool live = b < p.B && __ldg(p.bonus_tok + b) == -2;
    float best = -INFINITY;
    int best_idx = -1;
    const uint2 key = make_uint2(p.seed_lo, p.seed_hi);
    for (int t = 0; t < tiles.n_tiles; ++t) {
      int n0, nw;
      tiles.tile(t, n0, nw);
      const int buf = t & 1;
      mbar_wait(tmem_full + buf, (t >> 1) & 1u, p.dev_status);
      tc_fence_after();
      const int ncols = min(nw, p.V - n0);
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(warp * 32) << 16) + static_cast<uint32_t>(buf * SM_BN);
      if (__any_sync(0xffffffffu, live)) {
        for (int c0 = 0; c0 < ncols; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(taddr + c0, r);
          tc_wait_ld();
          if (live) {
#pragma unroll
            for (int j4 = 0; j4 < 32; j4 += 4) {
              const int v0 = n0 + c0 + j4;          // multiple of 4: one Philox call covers 4 columns
              const uint4 w = philox4x32_10(make_uint4(static_cast<unsigned>(v0 >> 2), static_cast<unsigned>(b),
                                                       p.step_lo, p.step_hi), key);
              const unsigned int ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                if (c0 + j4 + j < ncols) {
                  const float y = fmaf(__uint_as_float(r[j4 + j]), p.scale, gumbel_from_word(ww[j]));
                  if (y > best) { best = y; best_idx = v0 + j; }   // ascending v: ties keep the lowest index
                }
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tmem_empty + buf);
    }
    SamplePartial out;
    out.y = best; out.idx = best_idx;
    p.partial[static_cast<size_t>(range) * (p.n_mt * SM_BM) + b] = out;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------
// Few sequences (B <= 64): operands swapped. W is the M-side operand (128 vocabulary rows per
// MMA), the compact rows are the N side (16, 32 or 64 columns), so a pipeline stage is 16 KB of W
// plus 2-8 KB of Hc and the ring (9-12 stages) carries almost only W: enough bytes in
// flight to keep HBM busy, which the 128 x 256 tile above cannot do with its 48 KB stages.
// TMEM lane = vocabulary entry, column = sequence; each epilogue thread keeps a running best
// per sequence in registers and the CTA reduces them at the end. One group of four epilogue warps
// serves 32 sequence columns (64 columns: two groups, 320 threads); the loader and the MMA issuer
// are the two warps after the epilogue warps.
// ---------------------------------------------------------------------------------------
constexpr int SW_BM = 128, SW_BK = 64, SW_MAX_STAGES = 12, SW_MAX_SEQ = 32;   // SW_MAX_SEQ: sequences per epilogue group
constexpr int SW_MAX_GROUPS = 2, SW_TMEM_COLS = 128;
constexpr int SW_A_BYTES = SW_BM * SW_BK * 2;           // 16 KB of W per stage

struct SampleSwapParams {
  SampleParams base;
  int N;            // sequence columns: 16, 32 or 64
  int groups;       // epilogue warp groups: ceil(N / 32)
  int stages, stage_bytes;
};

template <int kGroups>
__global__ void __launch_bounds__((4 * kGroups + 2) * 32, 1)
sample_gemm_swapped_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_hc,
                           const SampleSwapParams sp) {
  pdl_launch_dependents();
  const SampleParams& p = sp.base;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base_u32 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base_u32 - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sp.stages * sp.stage_bytes);
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = bars + SW_MAX_STAGES;
  uint64_t* tmem_full = bars + 2 * SW_MAX_STAGES;
  uint64_t* tmem_empty = bars + 2 * SW_MAX_STAGES + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * SW_MAX_STAGES + 4);
  float* red_y = reinterpret_cast<float*>(bars + 2 * SW_MAX_STAGES + 6);    // [epilogue warps][32 sequences]
  int* red_i = reinterpret_cast<int*>(red_y + 4 * SW_MAX_GROUPS * SW_MAX_SEQ);
  constexpr int loader_warp = 4 * kGroups, issuer_warp = loader_warp + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int range = blockIdx.x;
  // vocabulary rows of this CTA: 128-row tiles of an equal share (in units of 16 rows)
  const int V16 = (p.V + 15) >> 4;
  const int u0 = static_cast<int>((static_cast<long long>(V16) * range) / p.n_ranges);
  const int u1 = static_cast<int>((static_cast<long long>(V16) * (range + 1)) / p.n_ranges);
  const int v_begin = u0 << 4, v_end = min(u1 << 4, p.V);
  const int n_tiles = (v_end - v_begin + SW_BM - 1) / SW_BM;
  const int n_kb = p.d / SW_BK;

  if (threadIdx.x == 0) {
    for (int i = 0; i < sp.stages; ++i) { mbar_init(full_bar + i, 1); mbar_init(empty_bar + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tmem_full + i, 1); mbar_init(tmem_empty + i, 4 * kGroups); }
    fence_mbar_init();
  }
  if (warp == issuer_warp) {
    tmem_alloc(tmem_slot, SW_TMEM_COLS);          // two accumulators of at most 64 columns
    tmem_relinquish();
  }
  if (warp == loader_warp && lane == 0) { prefetch_tmap(&tmap_hc); prefetch_tmap(&tmap_w); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();   // the compact rows come from the gather kernel

  if (warp == loader_warp) {
    if (lane == 0) {   // ---------------------------------------------------------- TMA producer
      int stage = 0;
      uint32_t phase = 0;
      const uint32_t tx = static_cast<uint32_t>(SW_A_BYTES + sp.N * SW_BK * 2);
      for (int t = 0; t < n_tiles; ++t) {
        for (int kb = 0; kb < n_kb; ++kb) {
          mbar_wait(empty_bar + stage, phase ^ 1u, p.dev_status);
          uint8_t* sa = smem + stage * sp.stage_bytes;
          mbar_expect_tx(full_bar + stage, tx);
          tma_load_2d(sa, &tmap_w, full_bar + stage, kb * SW_BK, v_begin + t * SW_BM);   // rows past V: zero fill
          tma_load_2d(sa + SW_A_BYTES, &tmap_hc, full_bar + stage, kb * SW_BK, 0);
          if (++stage == sp.stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == issuer_warp) {
    if (lane == 0) {   // ---------------------------------------------------------- MMA issuer
      int stage = 0;
      uint32_t phase = 0;
      const uint32_t idesc = idesc_bf16(SW_BM, sp.N, false, false);
      for (int t = 0; t < n_tiles; ++t) {
        const int buf = t & 1;
        mbar_wait(tmem_empty + buf, ((t >> 1) & 1u) ^ 1u, p.dev_status);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * 64);
        for (int kb = 0; kb < n_kb; ++kb) {
          mbar_wait(full_bar + stage, phase, p.dev_status);
          tc_fence_after();
          const uint32_t sa = base_u32 + stage * sp.stage_bytes;
          const uint64_t adesc = smem_desc_sw128(sa, 1024, 16);
          const uint64_t bdesc = smem_desc_sw128(sa + SW_A_BYTES, 1024, 16);
#pragma unroll
          for (int k = 0; k < SW_BK / 16; ++k) tc_mma_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | k) != 0);
          tc_commit(empty_bar + stage);
          if (++stage == sp.stages) { stage = 0; phase ^= 1u; }
        }
        tc_commit(tmem_full + buf);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (4 warps per 32 sequences)
    const int grp = warp >> 2, wq = warp & 3;     // sequence group, TMEM lane quarter
    const int b0 = grp * SW_MAX_SEQ;              // first sequence of this group
    const int row = wq * 32 + lane;               // TMEM lane = vocabulary entry of the tile
    unsigned int live_mask = 0;                   // bit j: sequence b0 + j wants a sample
    for (int j = 0; j < SW_MAX_SEQ && b0 + j < p.B; ++j)
      if (__ldg(p.bonus_tok + b0 + j) == -2) live_mask |= 1u << j;
    float best[SW_MAX_SEQ];
    int best_idx[SW_MAX_SEQ];
#pragma unroll
    for (int b = 0; b < SW_MAX_SEQ; ++b) { best[b] = -INFINITY; best_idx[b] = -1; }
    const uint2 key = make_uint2(p.seed_lo, p.seed_hi);
    for (int t = 0; t < n_tiles; ++t) {
      const int buf = t & 1;
      mbar_wait(tmem_full + buf, (t >> 1) & 1u, p.dev_status);
      tc_fence_after();
      uint32_t r[32];
      tmem_ld32(tmem_base + (static_cast<uint32_t>(wq * 32) << 16) + static_cast<uint32_t>(buf * 64 + b0), r);
      tc_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tmem_empty + buf);     // values are in registers: the buffer is free
      const int v = v_begin + t * SW_BM + row;
      if (v < v_end) {
#pragma unroll
        for (int b = 0; b < SW_MAX_SEQ; ++b) {
          if ((live_mask >> b) & 1u) {
            const uint4 w = philox4x32_10(make_uint4(static_cast<unsigned>(v >> 2), static_cast<unsigned>(b0 + b),
                                                     p.step_lo, p.step_hi), key);
            const unsigned int word = (v & 2) ? ((v & 1) ? w.w : w.z) : ((v & 1) ? w.y : w.x);
            const float y = fmaf(__uint_as_float(r[b]), p.scale, gumbel_from_word(word));
            if (y > best[b]) { best[b] = y; best_idx[b] = v; }   // ascending v: ties keep the lowest index
          }
        }
      }
    }
    // CTA-wide best per sequence: warp shuffles, then the four warps through shared memory
#pragma unroll
    for (int b = 0; b < SW_MAX_SEQ; ++b) {
      if (!((live_mask >> b) & 1u)) continue;     // uniform across the CTA
      float y = best[b];
      int i = best_idx[b];
      for (int o = 16; o > 0; o >>= 1) {
        const float oy = __shfl_xor_sync(0xffffffffu, y, o);
        const int oi = __shfl_xor_sync(0xffffffffu, i, o);
        if (oi >= 0 && (i < 0 || oy > y || (oy == y && oi < i))) { y = oy; i = oi; }
      }
      if (lane == 0) { red_y[warp * SW_MAX_SEQ + b] = y; red_i[warp * SW_MAX_SEQ + b] = i; }
    }
    asm volatile("bar.sync 2, %0;" ::"n"(128 * kGroups) : "memory");   // all epilogue warps
    if (wq == 0 && b0 + lane < p.B && ((live_mask >> lane) & 1u)) {
      float y = red_y[warp * SW_MAX_SEQ + lane];
      int i = red_i[warp * SW_MAX_SEQ + lane];
      for (int w2 = 1; w2 < 4; ++w2) {
        const float oy = red_y[(warp + w2) * SW_MAX_SEQ + lane];
        const int oi = red_i[(warp + w2) * SW_MAX_SEQ + lane];
        if (oi >= 0 && (i < 0 || oy > y || (oy == y && oi < i))) { y = oy; i = oi; }
      }
      SamplePartial out;
      out.y = y; out.idx = i;
      p.partial[static_cast<size_t>(range) * (p.n_mt * SM_BM) + b0 + lane] = out;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == issuer_warp) {
    tc_fence_after();
    tmem_dealloc(tmem_base, SW_TMEM_COLS);
  }
}

__global__ void __launch_bounds__(256)
sample_finalize_kernel(const SampleParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (b >= p.B) return;
  if (__ldg(p.bonus_tok + b) != -2) return;
  float best = -INFINITY;
  int idx = -1;
  for (int r = lane; r < p.n_ranges; r += 32) {
    const SamplePartial q = p.partial[static_cast<size_t>(r) * (p.n_mt * SM_BM) + b];
    if (q.idx >= 0 && (q.y > best || (q.y == best && q.idx < idx) || idx < 0)) { best = q.y; idx = q.idx; }
  }
  for (int o = 16; o > 0; o >>= 1) {
    const float oy = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (oi >= 0 && (idx < 0 || oy > best || (oy == best && oi < idx))) { best = oy; idx = oi; }
  }
  if (lane == 0) {
    p.bonus_tok[b] = idx;
    if (p.sample_value) p.sample_value[b] = best;
  }
}

static int sample_plan(const trispec_sample_args* a, int* n_mt, int* n_ranges) {
  if (!a || a->B <= 0 || a->T <= 0 || a->d <= 0 || a->V <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->T > 64 || (a->d % SM_BK) != 0) return TRISPEC_ERR_UNSUPPORTED;
  *n_mt = (a->B + SM_BM - 1) / SM_BM;
  int r = device_sm_count() / *n_mt;
  if (r < 1) r = 1;
  const int V16 = (a->V + 15) / 16;
  if (r > V16) r = V16;
  *n_ranges = r;
  return TRISPEC_OK;
}

}  // namespace trispec

extern "C" size_t trispec_sample_bonus_workspace(const trispec_sample_args* a) {
  using namespace trispec;
  int n_mt, n_ranges;
  if (sample_plan(a, &n_mt, &n_ranges) != TRISPEC_OK) return 0;
  const size_t hc = static_cast<size_t>(n_mt) * SM_BM * a->d * 2;
  const size_t part = static_cast<size_t>(n_ranges) * n_mt * SM_BM * sizeof(SamplePartial);
  return ((hc + 255) / 256) * 256 + part;
}

extern "C" int trispec_sample_bonus(const trispec_sample_args* a, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  int n_mt, n_ranges;
  int rc = sample_plan(a, &n_mt, &n_ranges);
  if (rc != TRISPEC_OK) return rc;
  if (!a->h || !a->W || !a->last_node || !a->bonus_tok || !a->workspace) return TRISPEC_ERR_INVALID_ARG;
  if (!aligned16(a->h) || !aligned16(a->W) || (reinterpret_cast<uintptr_t>(a->workspace) & 255u))
    return TRISPEC_ERR_INVALID_ARG;
  if (!(a->logit_scale > 0.f) || !isfinite(a->logit_scale)) return TRISPEC_ERR_INVALID_ARG;
  if (a->workspace_bytes < trispec_sample_bonus_workspace(a)) return TRISPEC_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  SampleParams p;
  p.B = a->B; p.T = a->T; p.d = a->d; p.V = a->V; p.n_mt = n_mt; p.n_ranges = n_ranges;
  p.scale = a->logit_scale;
  p.seed_lo = static_cast<unsigned int>(a->seed & 0xffffffffull); p.seed_hi = static_cast<unsigned int>(a->seed >> 32);
  p.step_lo = static_cast<unsigned int>(a->step & 0xffffffffull); p.step_hi = static_cast<unsigned int>(a->step >> 32);
  p.h = static_cast<const uint16_t*>(a->h);
  p.hc = static_cast<uint16_t*>(a->workspace);
  const size_t hc_bytes = ((static_cast<size_t>(n_mt) * SM_BM * a->d * 2 + 255) / 256) * 256;
  p.partial = reinterpret_cast<SamplePartial*>(static_cast<uint8_t*>(a->workspace) + hc_bytes);
  p.last_node = a->last_node; p.bonus_tok = a->bonus_tok; p.sample_value = a->sample_value;
  p.dev_status = a->dev_status;

  CUtensorMap tm_hc, tm_w;
  {
    const uint64_t dims[2] = {static_cast<uint64_t>(a->d), static_cast<uint64_t>(n_mt) * SM_BM};
    const uint64_t strides[1] = {static_cast<uint64_t>(a->d) * 2};
    const uint32_t box[2] = {SM_BK, 64};
    if (!cached_tmap_bf16(&tm_hc, p.hc, 2, dims, strides, box)) return TRISPEC_ERR_CUDA;
  }
  {
    const uint64_t dims[2] = {static_cast<uint64_t>(a->d), static_cast<uint64_t>(a->V)};
    const uint64_t strides[1] = {static_cast<uint64_t>(a->d) * 2};
    const uint32_t box[2] = {SM_BK, 64};
    if (!cached_tmap_bf16(&tm_w, a->W, 2, dims, strides, box)) return TRISPEC_ERR_CUDA;
  }
  TRISPEC_CUDA_OK(launch_dependent(sample_gather_kernel, static_cast<unsigned>(n_mt * SM_BM), 256, 0, st, 1, p));
  count_launch();
  if (a->B <= SW_MAX_SEQ * SW_MAX_GROUPS) {
    // few sequences: W on the M side, deep ring of small stages
    SampleSwapParams sp;
    sp.base = p;
    sp.N = a->B <= 16 ? 16 : (a->B <= 32 ? 32 : 64);
    sp.groups = (sp.N + SW_MAX_SEQ - 1) / SW_MAX_SEQ;
    sp.stage_bytes = SW_A_BYTES + sp.N * SW_BK * 2;
    sp.stages = (224 * 1024) / sp.stage_bytes;
    if (sp.stages > SW_MAX_STAGES) sp.stages = SW_MAX_STAGES;
    const int smem_bytes = sp.stages * sp.stage_bytes + 1024 + 3072;
    CUtensorMap tm_w128, tm_hcn;
    {
      const uint64_t dims[2] = {static_cast<uint64_t>(a->d), static_cast<uint64_t>(a->V)};
      const uint64_t strides[1] = {static_cast<uint64_t>(a->d) * 2};
      const uint32_t box[2] = {SW_BK, SW_BM};
      if (!cached_tmap_bf16(&tm_w128, a->W, 2, dims, strides, box)) return TRISPEC_ERR_CUDA;
    }
    {
      const uint64_t dims[2] = {static_cast<uint64_t>(a->d), static_cast<uint64_t>(n_mt) * SM_BM};
      const uint64_t strides[1] = {static_cast<uint64_t>(a->d) * 2};
      const uint32_t box[2] = {SW_BK, static_cast<uint32_t>(sp.N)};
      if (!cached_tmap_bf16(&tm_hcn, p.hc, 2, dims, strides, box)) return TRISPEC_ERR_CUDA;
    }
    typedef void (*SwapKernel)(CUtensorMap, CUtensorMap, SampleSwapParams);
    const SwapKernel kernel = sp.groups == 1 ? sample_gemm_swapped_kernel<1> : sample_gemm_swapped_kernel<2>;
    static bool smem_set_sw[2][64] = {};
    rc = ensure_smem_limit(reinterpret_cast<const void*>(kernel), 227 * 1024, smem_set_sw[sp.groups - 1]);
    if (rc != TRISPEC_OK) return rc;
    TRISPEC_CUDA_OK(launch_dependent(kernel, static_cast<unsigned>(n_ranges),
                                     static_cast<unsigned>((4 * sp.groups + 2) * 32),
                                     static_cast<size_t>(smem_bytes), st, 1, tm_w128, tm_hcn, sp));
    count_launch();
  } else {
    static bool smem_set[64] = {};
    rc = ensure_smem_limit(reinterpret_cast<const void*>(sample_gemm_kernel), SM_SMEM_BYTES, smem_set);
    if (rc != TRISPEC_OK) return rc;
    TRISPEC_CUDA_OK(launch_dependent(sample_gemm_kernel, static_cast<unsigned>(n_mt * n_ranges), SM_THREADS,
                                     SM_SMEM_BYTES, st, 1, tm_hc, tm_w, p));
    count_launch();
  }
  TRISPEC_CUDA_OK(launch_dependent(sample_finalize_kernel, static_cast<unsigned>((a->B + 7) / 8), 256, 0, st, 1, p));
  count_launch();
  return TRISPEC_OK;
}
