// LM head fused with per-row softmax statistics (distributions p_i of Eq. 5 reduced to what
// the margin rule of Eq. 8 and the acceptance test of Eq. 6 need). The [rows x V] logits
// never reach global memory: each CTA streams a slice of the vocabulary through
// tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory) and its epilogue keeps, per row, a
// running (max, sum of exponentials, top-1, top-2) in registers across all of its vocabulary
// tiles (and the sum the entropy needs, when the caller asks for the entropy). A small second
// kernel merges the per-slice partials and computes the drafted-token probabilities.
//
// GEMM kernel layout (two CTAs on two SMs work as a pair on one 256 x 256 tile)
//   M tile  = 256 rows = 4 sequence slots x 64 node slots, 128 rows per CTA of the pair
//             (T <= 64; missing nodes are zero-filled by the TMA out-of-bounds rule)
//   N tile  = 256 vocabulary entries, plus one narrower tile (a multiple of 32) for the rest of
//             the CTA pair's vocabulary range; each CTA loads one half of a tile
//   K block = 64 bf16 = one 128-byte swizzle row; 4 MMAs of K = 16 per block
//   Per k-block a CTA stages its own 128 rows of H (16 KB) and half of the W tile (16 KB):
//   32 KB for 128 x 256 x 64 multiply-adds per SM, against 48 KB when every SM works
//   alone. The pipeline is bound by how fast W tiles reach shared memory, so this is what
//   lifts the tensor-core duty cycle.
//   warps 0-3: epilogue (one TMEM lane = one row per thread), warp 4: TMA producer,
//   warp 5: TMEM owner; in the leader CTA (cluster rank 0) one of its threads issues the
//   MMAs of the pair. Accumulators are double-buffered in TMEM (2 x 256 columns per CTA)
//   so that the epilogue of tile i overlaps the MMAs of tile i + 1.
//   Pair c works on M tile (c % n_mt) and vocabulary range (c / n_mt): pairs that share a
//   vocabulary range are neighbours and stream the same W tiles at the same time, so W is
//   read from HBM once and re-hit in L2.
//   Barriers: `full` lives in the leader and counts the bytes of both CTAs' loads; `empty`
//   and `tmem_full` exist in both CTAs and are signalled by the leader's commits;
//   `tmem_empty` lives in the leader and collects the epilogue warps of both CTAs.
#include <math.h>

#include <mutex>

#include "host_common.h"
#include "sm100.cuh"

namespace trispec {

constexpr int LM_BM = 128;                      // rows per CTA
constexpr int LM_BN = 256;
constexpr int LM_BK = 64;
constexpr int LM_STAGES = 6;
constexpr int LM_A_BYTES = LM_BM * LM_BK * 2;         // 16 KB
constexpr int LM_B_BYTES = (LM_BN / 2) * LM_BK * 2;   // 16 KB: this CTA's half of the W tile
constexpr int LM_BOX_BYTES = 64 * LM_BK * 2;    // one TMA box: 64 rows x 64 k
constexpr int LM_STAGE_BYTES = LM_A_BYTES + LM_B_BYTES;
constexpr int LM_THREADS = 192;
constexpr int LM_SMEM_BYTES = LM_STAGES * LM_STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr float kLog2e = 1.4426950408889634f;

struct __align__(16) LmPartial {
  float m, s, v1, v2;  // raw (unscaled) running max, sum of 2^((z-m)c), top-1 / top-2 raw logits
  int i1, i2;
  float t;             // sum of 2^((z-m)c) * z over the range (for the entropy: H = lse - E_p[z])
  int pad;
};

struct LmParams {
  int T, d, V;
  int n_seq;      // active sequences
  int n_mt;       // M tiles of 4 sequence slots = ceil(n_seq / 4)
  int n_ranges;   // vocabulary ranges of the main part: pair c < n_mt * n_ranges works on M tile c % n_mt, range c / n_mt
  int n_tail;     // pairs beyond those: each sweeps ALL M tiles over its slice of the vocabulary's tail
  int main_units; // 32-column units [0, main_units) belong to the main part, the rest to the tail
  float c;        // logit_scale * log2(e)
  const int32_t* seq_index;
  LmPartial* partial;  // [n_ranges + n_tail][n_mt * 256]
  int32_t* dev_status;
};

// Vocabulary range r of n_ranges, cut into tiles of 256 columns plus one narrower tile for the
// rest; all boundaries are multiples of 32 columns so that each CTA of a pair takes a half that
// is a multiple of 16. (A tile of 224 columns costs as much as one of 256 - its k-loop is as long
// and the MMA time does not shrink in proportion - so the rest is not spread over the tiles.)
struct TileIter {
  int u0, units, n_tiles;
  // part r of n_parts of the 32-column units [first, first + count)
  __device__ TileIter(int first, int count, int n_parts, int r) {
    // Every part gets count / n_parts units. What is left over goes to the first parts in chunks that
    // cost as few extra tiles as possible: a tile costs a whole k-loop whatever its width, so a chunk
    // first fills up a part's last, partial tile (no extra tile), and where the parts consist of whole
    // tiles it is a whole tile (few parts run one tile longer, instead of many).
    const int base = count / n_parts, rem = count - base * n_parts;
    const int chunk = 8 - (base & 7);               // 1..8
    u0 = first + r * base + min(rem, r * chunk);
    units = base + min(chunk, max(0, rem - r * chunk));
    n_tiles = (units + 7) >> 3;
  }
  __device__ void tile(int t, int& n0, int& nw) const {
    n0 = (u0 + 8 * t) << 5;
    nw = min(8, units - 8 * t) << 5;
  }
};

// What a CTA pair works on. A main pair computes one M tile over one vocabulary range (one sweep). When
// the M tiles do not divide the pairs of the chip, the pairs left over take the tail of the vocabulary:
// each of them sweeps all M tiles, one after the other, over its own slice of that tail, which is
// short enough to stay in L2 between the sweeps; the main ranges shrink accordingly, so that every
// pair of the chip runs about the same number of tiles.
struct PairWork {
  int n_sweeps, mt0, part;      // M tile of sweep s = mt0 + s; `part` = row block of the partial array
  TileIter tiles;
  __device__ PairWork(const LmParams& p, int pair)
      : n_sweeps(1), mt0(0), part(0), tiles(0, 0, 1, 0) {
    const int V32 = (p.V + 31) >> 5;
    const int n_main = p.n_mt * p.n_ranges;
    if (pair < n_main) {
      mt0 = pair % p.n_mt;
      part = pair / p.n_mt;
      tiles = TileIter(0, p.main_units, p.n_ranges, part);
    } else {
      n_sweeps = p.n_mt;
      part = p.n_ranges + (pair - n_main);
      tiles = TileIter(p.main_units, V32 - p.main_units, p.n_tail, pair - n_main);
    }
  }
};

template <bool kEntropy>
__global__ void __launch_bounds__(LM_THREADS, 1)
lmhead_gemm_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_w,
                   const LmParams p) {
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  // the dynamic window starts at the same offset in both CTAs of the pair, so the aligned
  // layouts coincide, as the paired MMA requires
  const uint32_t base_u32 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base_u32 - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + LM_STAGES * LM_STAGE_BYTES);
  uint64_t* full_bar = bars;                      // [LM_STAGES]  (used in the leader)
  uint64_t* empty_bar = bars + LM_STAGES;         // [LM_STAGES]
  uint64_t* tmem_full = bars + 2 * LM_STAGES;     // [2]
  uint64_t* tmem_empty = bars + 2 * LM_STAGES + 2;  // [2]        (used in the leader)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * LM_STAGES + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();        // 0 = leader
  const int pair = blockIdx.x >> 1;
  const PairWork work(p, pair);
  const TileIter& tiles = work.tiles;
  const int n_kb = p.d / LM_BK;

  if (threadIdx.x == 0) {
    for (int i = 0; i < LM_STAGES; ++i) { mbar_init(full_bar + i, 1); mbar_init(empty_bar + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tmem_full + i, 1); mbar_init(tmem_empty + i, 8); }
    fence_mbar_init();
  }
  if (warp == 5) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  if (warp == 4 && lane == 0) { prefetch_tmap(&tmap_h); prefetch_tmap(&tmap_w); }
  tc_fence_before();
  cluster_sync_all();                             // both CTAs' barriers and TMEM are ready
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      // sequence slots of this CTA; a slot past the last active sequence re-reads the M tile's
      // first sequence (its rows are computed and never looked at), which keeps the byte count
      // of a stage the same in both CTAs
      int stage = 0;
      uint32_t phase = 0;
      for (int sweep = 0; sweep < work.n_sweeps; ++sweep) {
      const int a_first = 4 * (work.mt0 + sweep);
      int a0 = a_first + 2 * static_cast<int>(rank), a1 = a0 + 1;
      if (a0 >= p.n_seq) a0 = a_first;
      if (a1 >= p.n_seq) a1 = a_first;
      const int s0 = p.seq_index ? __ldg(p.seq_index + a0) : a0;
      const int s1 = p.seq_index ? __ldg(p.seq_index + a1) : a1;
      for (int t = 0; t < tiles.n_tiles; ++t) {
        int n0, nw;
        tiles.tile(t, n0, nw);
        const int nh = nw >> 1;                   // rows of W this CTA stages
        const int nbox = (nh + 63) >> 6;
        const int w0 = n0 + static_cast<int>(rank) * nh;
        const uint32_t tx_pair = 2u * static_cast<uint32_t>(2 + nbox) * LM_BOX_BYTES;
        for (int kb = 0; kb < n_kb; ++kb) {
          mbar_wait(empty_bar + stage, phase ^ 1u, p.dev_status);
          uint8_t* sa = smem + stage * LM_STAGE_BYTES;
          uint8_t* sb = sa + LM_A_BYTES;
          if (rank == 0) mbar_expect_tx(full_bar + stage, tx_pair);
          const uint32_t fb = cluster_map(smem_u32(full_bar + stage), 0);
          tma_load_3d_pair(sa, &tmap_h, fb, kb * LM_BK, 0, s0);
          tma_load_3d_pair(sa + LM_BOX_BYTES, &tmap_h, fb, kb * LM_BK, 0, s1);
          for (int j = 0; j < nbox; ++j)
            tma_load_2d_pair(sb + j * LM_BOX_BYTES, &tmap_w, fb, kb * LM_BK, w0 + 64 * j);
          if (++stage == LM_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      }   // sweeps
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA)
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      const int n_all = work.n_sweeps * tiles.n_tiles;      // the accumulator buffers alternate over all sweeps
      for (int tt = 0; tt < n_all; ++tt) {
        const int t = tt % tiles.n_tiles;
        int n0, nw;
        tiles.tile(t, n0, nw);
        const int buf = tt & 1;
        mbar_wait(tmem_empty + buf, ((tt >> 1) & 1u) ^ 1u, p.dev_status);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * LM_BN);
        const uint32_t idesc = idesc_bf16(2 * LM_BM, nw, false, false);
        for (int kb = 0; kb < n_kb; ++kb) {
          mbar_wait(full_bar + stage, phase, p.dev_status);
          tc_fence_after();
          const uint32_t sa = base_u32 + stage * LM_STAGE_BYTES;
          const uint64_t adesc = smem_desc_sw128(sa, 1024, 16);
          const uint64_t bdesc = smem_desc_sw128(sa + LM_A_BYTES, 1024, 16);
#pragma unroll
          for (int k = 0; k < LM_BK / 16; ++k) {
            // advancing 16 elements (32 bytes) along K inside the swizzle row: +2 in the
            // 16-byte-granular start address field
            tc_mma_ss_pair(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | k) != 0);
          }
          tc_commit_pair(empty_bar + stage, 3);   // the stage is free again in both CTAs
          if (++stage == LM_STAGES) { stage = 0; phase ^= 1u; }
        }
        tc_commit_pair(tmem_full + buf, 3);       // both CTAs' accumulators are complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3)
    const int row = warp * 32 + lane;  // TMEM lane == row of this CTA's half of the M tile
    const float c = p.c;
    const uint32_t tmem_empty_leader = cluster_map(smem_u32(tmem_empty), 0);
    for (int sweep = 0; sweep < work.n_sweeps; ++sweep) {
    float m = -INFINITY, s = 0.f, tz = 0.f, v1 = -INFINITY, v2 = -INFINITY;
    int i1 = -1, i2 = -1;
    for (int t = 0; t < tiles.n_tiles; ++t) {
      int n0, nw;
      tiles.tile(t, n0, nw);
      const int tt = sweep * tiles.n_tiles + t;
      const int buf = tt & 1;
      mbar_wait(tmem_full + buf, (tt >> 1) & 1u, p.dev_status);
      tc_fence_after();
      const int ncols = min(nw, p.V - n0);  // valid columns of this tile
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(warp * 32) << 16) + static_cast<uint32_t>(buf * LM_BN);
      for (int c0 = 0; c0 < ncols; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(taddr + c0, r);
        tc_wait_ld();
        const int nv = ncols - c0;  // >= 1
        float cmax = -INFINITY;
        if (nv >= 32) {
          // whole chunk valid: three-input max and packed fp32 pairs halve the instruction count
          float cm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            cm[0] = fmax3(cm[0], __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
            cm[1] = fmax3(cm[1], __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
            cm[2] = fmax3(cm[2], __uint_as_float(r[j + 4]), __uint_as_float(r[j + 5]));
            cm[3] = fmax3(cm[3], __uint_as_float(r[j + 6]), __uint_as_float(r[j + 7]));
          }
          cmax = fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3]));
          if (cmax > m) {
            const float f = ex2f((m - cmax) * c);
            s *= f;
            tz *= f;
            m = cmax;
          }
          const float nmc = -m * c;
          const float2 c2 = make_float2(c, c), nmc2 = make_float2(nmc, nmc);
          float2 acc2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
          float2 acz2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const float2 z = make_float2(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
            const float2 x = ffma2(z, c2, nmc2);
            const float2 e = make_float2(ex2f(x.x), ex2f(x.y));
            acc2[(j >> 1) & 1] = fadd2(acc2[(j >> 1) & 1], e);
            if (kEntropy) acz2[(j >> 1) & 1] = ffma2(e, z, acz2[(j >> 1) & 1]);
          }
          s += (acc2[0].x + acc2[0].y) + (acc2[1].x + acc2[1].y);
          if (kEntropy) tz += (acz2[0].x + acz2[0].y) + (acz2[1].x + acz2[1].y);
        } else {
          // ragged end of the vocabulary: columns past V count as -inf
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            float v = __uint_as_float(r[j]);
            if (j >= nv) { v = -INFINITY; r[j] = __float_as_uint(v); }
            cmax = fmaxf(cmax, v);
          }
          if (cmax > m) {
            const float f = ex2f((m - cmax) * c);
            s *= f;
            tz *= f;
            m = cmax;
          }
          const float mc = m * c;
          float acc = 0.f, acz = 0.f;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float e = ex2f(fmaf(__uint_as_float(r[j]), c, -mc));
            acc += e;
            // masked columns hold -inf with e = 0: keep 0 * inf out of the sum
            if (kEntropy) acz = fmaf(e, (j < nv) ? __uint_as_float(r[j]) : 0.f, acz);
          }
          s += acc;
          tz += acz;
        }
        if (cmax > v2) {
          const int col0 = n0 + c0;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float v = __uint_as_float(r[j]);
            if (v > v1) { v2 = v1; i2 = i1; v1 = v; i1 = col0 + j; }
            else if (v > v2) { v2 = v; i2 = col0 + j; }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tmem_empty_leader + static_cast<uint32_t>(buf) * 8u);
    }
    if (sweep == 0) pdl_wait();   // the partials of the previous pass may still be read until earlier kernels are done
    LmPartial out;
    out.m = m; out.s = s; out.v1 = v1; out.v2 = v2; out.i1 = i1; out.i2 = i2; out.t = tz; out.pad = 0;
    p.partial[static_cast<size_t>(work.part) * (p.n_mt * 2 * LM_BM) + ((work.mt0 + sweep) * 2 + rank) * LM_BM + row] = out;
    }   // sweeps
  }

  pdl_wait();
  // nobody leaves, and tensor memory stays allocated, until both CTAs are done: the leader's
  // MMAs write the peer's tensor memory and its commits arrive on the peer's barriers
  tc_fence_before();
  cluster_sync_all();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------
// Merge of the per-range partials + drafted-token logits.
// ---------------------------------------------------------------------------------------
struct LmFinalizeParams {
  int T, d, V, n_mt, n_ranges;
  int stride;       // partial rows per vocabulary range
  float scale, c;
  const int32_t* seq_index;
  const LmPartial* partial;
  const uint16_t *h, *W;
  const int32_t *parent, *tok;
  trispec_stats out;
};

constexpr int LM_FIN_THREADS = 256;   // 8 warps = 8 rows per block

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// larger value first, lower index on ties; index -1 marks "no entry"
__device__ __forceinline__ bool lm_better(float va, int ia, float vb, int ib) {
  return ia >= 0 && (ib < 0 || va > vb || (va == vb && ia < ib));
}
__device__ __forceinline__ void lm_top2_insert(float v, int i, float& v1, int& i1, float& v2, int& i2) {
  if (i < 0) return;
  if (lm_better(v, i, v1, i1)) { v2 = v1; i2 = i1; v1 = v; i1 = i; }
  else if (lm_better(v, i, v2, i2)) { v2 = v; i2 = i; }
}

// running (max, sum of exponentials, sum of exponentials x logit) of a set of vocabulary ranges
struct LmRowAcc { float m, s, t; };
__device__ __forceinline__ void lm_fold(LmRowAcc& a, float m, float s, float t, float c) {
  const float M = fmaxf(a.m, m);
  const float fa = (a.m == -INFINITY) ? 0.f : ex2f((a.m - M) * c);
  const float fb = (m == -INFINITY) ? 0.f : ex2f((m - M) * c);
  a.s = a.s * fa + s * fb;
  a.t = a.t * fa + t * fb;
  a.m = M;
}

// One warp per (active sequence, node): merges the row's partial statistics and, for a child
// node, computes the logit of its drafted token in its parent's row (a d-long dot product).
// The dot product needs only the kernel's inputs, so it runs before the wait for the GEMM and
// overlaps that kernel's tail; after the wait every lane loads its share of the partials of
// the node's row and of the parent's row in one go and the warp folds them by shuffles.
__global__ void __launch_bounds__(LM_FIN_THREADS)
lmhead_finalize_kernel(const LmFinalizeParams p, int n_seq) {
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31;
  const long long w = static_cast<long long>(blockIdx.x) * (LM_FIN_THREADS / 32) + (threadIdx.x >> 5);
  const int T = p.T;
  const bool active = w < static_cast<long long>(n_seq) * T;
  const int a = active ? static_cast<int>(w / T) : 0, node = active ? static_cast<int>(w % T) : 0;
  const int seq = p.seq_index ? __ldg(p.seq_index + a) : a;
  const long long row0 = static_cast<long long>(seq) * T;

  // ---- drafted-token logit z[parent(node)][tok[node]]: inputs only
  bool has_draft = false;
  int par = 0;
  float dot = 0.f;
  if (active && node >= 1) {
    par = __ldg(p.parent + row0 + node);
    const int tk = __ldg(p.tok + row0 + node);
    has_draft = par >= 0 && par < node && tk >= 0 && tk < p.V;
    if (has_draft) {
      const uint4* hv = reinterpret_cast<const uint4*>(p.h + (row0 + par) * p.d);
      const uint4* wv = reinterpret_cast<const uint4*>(p.W + static_cast<long long>(tk) * p.d);
      float acc[2] = {0.f, 0.f};
#pragma unroll 4
      for (int i = lane; i < p.d / 8; i += 32) {
        const uint4 x = __ldg(hv + i), y = __ldg(wv + i);
        acc[0] = fmaf(bf16_lo(x.x), bf16_lo(y.x), acc[0]); acc[1] = fmaf(bf16_hi(x.x), bf16_hi(y.x), acc[1]);
        acc[0] = fmaf(bf16_lo(x.y), bf16_lo(y.y), acc[0]); acc[1] = fmaf(bf16_hi(x.y), bf16_hi(y.y), acc[1]);
        acc[0] = fmaf(bf16_lo(x.z), bf16_lo(y.z), acc[0]); acc[1] = fmaf(bf16_hi(x.z), bf16_hi(y.z), acc[1]);
        acc[0] = fmaf(bf16_lo(x.w), bf16_lo(y.w), acc[0]); acc[1] = fmaf(bf16_hi(x.w), bf16_hi(y.w), acc[1]);
      }
      dot = acc[0] + acc[1];
      for (int o2 = 16; o2 > 0; o2 >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o2);
    }
  }
  if (!has_draft) par = node;                    // a valid row to load; the result is not used

  pdl_wait();                                    // the partials come from the GEMM kernel
  if (!active) return;

  // ---- merge of the per-range partials: own row (all statistics) and parent row (max, sum)
  const size_t stride = static_cast<size_t>(p.stride);
  const LmPartial* own = p.partial + static_cast<size_t>(a) * 64 + node;
  const LmPartial* parp = p.partial + static_cast<size_t>(a) * 64 + par;
  LmRowAcc ro = {-INFINITY, 0.f, 0.f}, rp = {-INFINITY, 0.f, 0.f};
  float v1 = -INFINITY, v2 = -INFINITY;
  int i1 = -1, i2 = -1;
  for (int r0 = 0; r0 < p.n_ranges; r0 += 96) {  // three ranges per lane and round, loads first
    float4 qa[3], qb[3];
    float2 qp[3];
#pragma unroll
    for (int u = 0; u < 3; ++u) {
      const int r = r0 + lane + 32 * u;
      qa[u] = make_float4(-INFINITY, 0.f, -INFINITY, -INFINITY);
      qb[u] = make_float4(__int_as_float(-1), __int_as_float(-1), 0.f, 0.f);
      qp[u] = make_float2(-INFINITY, 0.f);
      if (r < p.n_ranges) {
        const float4* q4 = reinterpret_cast<const float4*>(own + r * stride);
        qa[u] = q4[0];                           // m, s, v1, v2
        qb[u] = q4[1];                           // i1, i2, t, pad
        qp[u] = *reinterpret_cast<const float2*>(parp + r * stride);   // m, s of the parent's row
      }
    }
#pragma unroll
    for (int u = 0; u < 3; ++u) {
      lm_fold(ro, qa[u].x, qa[u].y, qb[u].z, p.c);
      lm_fold(rp, qp[u].x, qp[u].y, 0.f, p.c);
      lm_top2_insert(qa[u].z, __float_as_int(qb[u].x), v1, i1, v2, i2);
      lm_top2_insert(qa[u].w, __float_as_int(qb[u].y), v1, i1, v2, i2);
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    lm_fold(ro, __shfl_xor_sync(0xffffffffu, ro.m, o), __shfl_xor_sync(0xffffffffu, ro.s, o),
            __shfl_xor_sync(0xffffffffu, ro.t, o), p.c);
    lm_fold(rp, __shfl_xor_sync(0xffffffffu, rp.m, o), __shfl_xor_sync(0xffffffffu, rp.s, o), 0.f, p.c);
    const float ov1 = __shfl_xor_sync(0xffffffffu, v1, o), ov2 = __shfl_xor_sync(0xffffffffu, v2, o);
    const int oi1 = __shfl_xor_sync(0xffffffffu, i1, o), oi2 = __shfl_xor_sync(0xffffffffu, i2, o);
    lm_top2_insert(ov1, oi1, v1, i1, v2, i2);
    lm_top2_insert(ov2, oi2, v1, i1, v2, i2);
  }
  if (lane == 0) {
    const float lse = ro.m * p.scale + logf(ro.s);
    const long long o = row0 + node;
    p.out.max[o] = ro.m * p.scale;
    p.out.lse[o] = lse;
    p.out.top1_val[o] = v1 * p.scale;
    p.out.top2_val[o] = v2 * p.scale;
    p.out.top1_idx[o] = i1;
    p.out.top2_idx[o] = i2;
    p.out.p_top1[o] = expf(v1 * p.scale - lse);
    p.out.p_top2[o] = expf(v2 * p.scale - lse);
    // entropy in nats: H = lse - E_p[z], E_p[z] = scale * sum(e * z_raw) / sum(e); never below 0
    if (p.out.entropy) p.out.entropy[o] = fmaxf(lse - p.scale * (ro.t / ro.s), 0.f);
    float dl = __int_as_float(0x7fc00000), pd = dl;
    if (has_draft) {
      dl = dot * p.scale;
      pd = expf(dl - (rp.m * p.scale + logf(rp.s)));
    }
    p.out.draft_logit[o] = dl;
    p.out.p_draft[o] = pd;
  }
}

// ---------------------------------------------------------------------------------------
// One sequence (batch-1 decoding, the paper's own setting): operands swapped. With at most 64
// rows the GEMM is bound by streaming W, and the pair kernel above spends half of its ring
// on H tiles. Here W is the M-side operand (128 vocabulary entries per MMA), the sequence's
// rows are the N side (16-64 columns), one CTA per SM, and a stage is KPS k-blocks of 16 KB of W plus
// 2-8 KB of H each, almost all of it W. TMEM lane = vocabulary entry, column = tree node.
// A CTA's vocabulary range is a multiple of 16 entries but rarely of 128: its last tile is fetched with
// a second, lower box (only the rows the range owns; the MMA still spans 128 lanes, the lanes past
// the range read stale shared memory and are ignored), so the chip streams W once, not the 5-18 %
// more that whole tiles would cost on a launch that is bound by exactly this stream.
// With KPS = 4 (any vocabulary that is a multiple of 8) W is read through a 4-D view
// [V/8][d/64][8 rows][64 elements], whose box puts the k-blocks of one group of 8 rows next to each
// other in the request stream; the stage then holds [16 row groups][KPS k-blocks][8 rows][128 B], and
// the MMA descriptor of k-block j starts j KB in with KPS KB between row groups. KPS = 1 is the
// plain 2-D view, the same layout with one k-block.
// Epilogue: per tile a warp reduces 32 columns at once over its 32 vocabulary entries with
// transposing shuffle butterflies (top-2 with indices, then the sums of exponentials), after which
// lane l holds column l's result and folds it into the running statistics it keeps for that column.
// ---------------------------------------------------------------------------------------
constexpr int LW_BM = 128, LW_BK = 64, LW_MAX_STAGES = 12, LW_THREADS = 192;
constexpr int LW_A_BYTES = LW_BM * LW_BK * 2;           // 16 KB of W per stage
constexpr int LW_ROWS = 64;                              // partial rows per vocabulary range

struct LmRowsParams {
  LmParams base;
  int N;            // node columns: T rounded up to 16
  int stages, stage_bytes;
  int tail_rows;    // height of the second W box (a multiple of 16 below 128), 0 = no second box
};

struct LmColStats { float m, s, t, v1, v2; int i1, i2; };

// One 32-column chunk of a tile in the epilogue of lmhead_rows_kernel: r[j] = logit of column col0 + j at this
// lane's vocabulary entry my_v. Per column: top-2 (value, vocabulary index) and the sum of exponentials over
// the warp's 32 vocabulary entries, folded into the running statistics `run` of column col0 + lane. A
// transposing butterfly does all columns at once: in the step with distance o a lane keeps half of the
// columns it still holds, hands the other half to its partner and merges what it receives, so that after
// the steps lane l holds column l. NC = 32 columns take five steps; when the tree has at most 16 nodes
// (NC = 16: chains), four steps leave lanes l and l + 16 with column l over one half of the entries each,
// and one more exchange merges the halves (lanes 16-31 then hold copies, which nothing reads).
template <bool kEntropy, int NC>
__device__ __forceinline__ void lm_rows_chunk_nc(const uint32_t (&r)[32], bool valid, int my_v, int col0, int N, int lane,
                                                 float c, LmColStats& run) {
  float v1[NC], v2[NC];
  int i1[NC], i2[NC];
#pragma unroll
  for (int j = 0; j < NC; ++j) {
    const bool on = valid && (col0 + j < N);
    v1[j] = on ? __uint_as_float(r[j]) : -INFINITY;
    i1[j] = on ? my_v : -1;
    v2[j] = -INFINITY;
    i2[j] = -1;
  }
#pragma unroll
  for (int o = NC / 2; o > 0; o >>= 1) {
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < o; ++i) {
      const float sv1 = up ? v1[i] : v1[i + o], sv2 = up ? v2[i] : v2[i + o];
      const int si1 = up ? i1[i] : i1[i + o], si2 = up ? i2[i] : i2[i + o];
      float kv1 = up ? v1[i + o] : v1[i], kv2 = up ? v2[i + o] : v2[i];
      int ki1 = up ? i1[i + o] : i1[i], ki2 = up ? i2[i + o] : i2[i];
      const float rv1 = __shfl_xor_sync(0xffffffffu, sv1, o), rv2 = __shfl_xor_sync(0xffffffffu, sv2, o);
      const int ri1 = __shfl_xor_sync(0xffffffffu, si1, o), ri2 = __shfl_xor_sync(0xffffffffu, si2, o);
      lm_top2_insert(rv1, ri1, kv1, ki1, kv2, ki2);
      lm_top2_insert(rv2, ri2, kv1, ki1, kv2, ki2);
      v1[i] = kv1; v2[i] = kv2; i1[i] = ki1; i2[i] = ki2;
    }
  }
  if (NC == 16) {   // lanes l and l ^ 16 hold the same column over different vocabulary entries
    const float rv1 = __shfl_xor_sync(0xffffffffu, v1[0], 16), rv2 = __shfl_xor_sync(0xffffffffu, v2[0], 16);
    const int ri1 = __shfl_xor_sync(0xffffffffu, i1[0], 16), ri2 = __shfl_xor_sync(0xffffffffu, i2[0], 16);
    lm_top2_insert(rv1, ri1, v1[0], i1[0], v2[0], i2[0]);
    lm_top2_insert(rv2, ri2, v1[0], i1[0], v2[0], i2[0]);
  }
  const float m_t = v1[0];                  // this lane's column: col0 + (lane mod NC)
  // every lane needs every column's maximum for its exponentials
  float es[NC], et[NC];
#pragma unroll
  for (int j = 0; j < NC; ++j) {
    const float mj = __shfl_sync(0xffffffffu, m_t, j);
    const bool on = valid && (col0 + j < N);
    const float z = __uint_as_float(r[j]);
    es[j] = on ? ex2f((z - mj) * c) : 0.f;
    et[j] = (kEntropy && on) ? es[j] * z : 0.f;
  }
#pragma unroll
  for (int o = NC / 2; o > 0; o >>= 1) {
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < o; ++i) {
      const float ss = up ? es[i] : es[i + o], ks = up ? es[i + o] : es[i];
      es[i] = ks + __shfl_xor_sync(0xffffffffu, ss, o);
      if (kEntropy) {
        const float st2 = up ? et[i] : et[i + o], kt = up ? et[i + o] : et[i];
        et[i] = kt + __shfl_xor_sync(0xffffffffu, st2, o);
      }
    }
  }
  if (NC == 16) {
    es[0] += __shfl_xor_sync(0xffffffffu, es[0], 16);
    if (kEntropy) et[0] += __shfl_xor_sync(0xffffffffu, et[0], 16);
  }
  // fold the tile's statistics of this lane's column into the running ones
  LmRowAcc a = {run.m, run.s, run.t};
  lm_fold(a, m_t, es[0], et[0], c);
  run.m = a.m; run.s = a.s; run.t = a.t;
  lm_top2_insert(v1[0], i1[0], run.v1, run.i1, run.v2, run.i2);
  lm_top2_insert(v2[0], i2[0], run.v1, run.i1, run.v2, run.i2);
}
template <bool kEntropy>
__device__ __forceinline__ void lm_rows_chunk(const uint32_t (&r)[32], bool valid, int my_v, int col0, int N, int lane,
                                              float c, LmColStats& run) {
  if (N <= 16) lm_rows_chunk_nc<kEntropy, 16>(r, valid, my_v, col0, N, lane, c, run);
  else lm_rows_chunk_nc<kEntropy, 32>(r, valid, my_v, col0, N, lane, c, run);
}


template <bool kEntropy, int KPS>
__global__ void __launch_bounds__(LW_THREADS, 1)
lmhead_rows_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_wt,
                   const __grid_constant__ CUtensorMap tmap_h, const LmRowsParams sp) {
  pdl_launch_dependents();
  const LmParams& p = sp.base;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base_u32 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base_u32 - smem_u32(smem_raw));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + sp.stages * sp.stage_bytes);
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = bars + LW_MAX_STAGES;
  uint64_t* tmem_full = bars + 2 * LW_MAX_STAGES;
  uint64_t* tmem_empty = bars + 2 * LW_MAX_STAGES + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * LW_MAX_STAGES + 4);
  LmColStats* red = reinterpret_cast<LmColStats*>(bars + 2 * LW_MAX_STAGES + 6);   // [4 warps][64 columns]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int range = blockIdx.x;
  const int V16 = (p.V + 15) >> 4;
  const int u0 = static_cast<int>((static_cast<long long>(V16) * range) / p.n_ranges);
  const int u1 = static_cast<int>((static_cast<long long>(V16) * (range + 1)) / p.n_ranges);
  const int v_begin = u0 << 4, v_end = min(u1 << 4, p.V);
  const int n_tiles = (v_end - v_begin + LW_BM - 1) / LW_BM;
  const int n_kb = p.d / LW_BK;

  if (threadIdx.x == 0) {
    for (int i = 0; i < sp.stages; ++i) { mbar_init(full_bar + i, 1); mbar_init(empty_bar + i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(tmem_full + i, 1); mbar_init(tmem_empty + i, 4); }
    fence_mbar_init();
  }
  if (warp == 5) {
    tmem_alloc(tmem_slot, 128);                   // two accumulators of at most 64 columns
    tmem_relinquish();
  }
  if (warp == 4 && lane == 0) { prefetch_tmap(&tmap_h); prefetch_tmap(&tmap_w); prefetch_tmap(&tmap_wt); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4) {
    if (lane == 0) {   // ---------------------------------------------------------- TMA producer
      int stage = 0;
      uint32_t phase = 0;
      const int seq = p.seq_index ? __ldg(p.seq_index) : 0;     // the one active sequence
      const int h_bytes = sp.N * LW_BK * 2;
      for (int t = 0; t < n_tiles; ++t) {
        const int row0 = v_begin + t * LW_BM;
        // a box always delivers its full size (rows past V, k-blocks past d: zero fill)
        const bool low = sp.tail_rows > 0 && v_end - row0 <= sp.tail_rows;
        const CUtensorMap* tw = low ? &tmap_wt : &tmap_w;
        const int w_bytes = KPS * (low ? sp.tail_rows : LW_BM) * LW_BK * 2;
        for (int kb = 0; kb < n_kb; kb += KPS) {
          const int kc = min(KPS, n_kb - kb);
          mbar_wait(empty_bar + stage, phase ^ 1u, p.dev_status);
          uint8_t* sa = smem + stage * sp.stage_bytes;
          mbar_expect_tx(full_bar + stage, static_cast<uint32_t>(w_bytes + kc * h_bytes));
          if (KPS == 1) tma_load_2d(sa, tw, full_bar + stage, kb * LW_BK, row0);
          else tma_load_4d(sa, tw, full_bar + stage, 0, 0, kb, row0 >> 3);
          for (int j = 0; j < kc; ++j)                                                     // nodes past T: zero fill
            tma_load_3d(sa + KPS * LW_A_BYTES + j * h_bytes, &tmap_h, full_bar + stage, (kb + j) * LW_BK, 0, seq);
          if (++stage == sp.stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {   // ---------------------------------------------------------- MMA issuer
      int stage = 0;
      uint32_t phase = 0;
      const uint32_t idesc = idesc_bf16(LW_BM, sp.N, false, false);
      for (int t = 0; t < n_tiles; ++t) {
        const int buf = t & 1;
        mbar_wait(tmem_empty + buf, ((t >> 1) & 1u) ^ 1u, p.dev_status);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * 64);
        for (int kb = 0; kb < n_kb; kb += KPS) {
          const int kc = min(KPS, n_kb - kb);
          mbar_wait(full_bar + stage, phase, p.dev_status);
          tc_fence_after();
          const uint32_t sa = base_u32 + stage * sp.stage_bytes;
          for (int j = 0; j < kc; ++j) {
            const uint64_t adesc = smem_desc_sw128(sa + j * 1024, KPS * 1024, 16);
            const uint64_t bdesc = smem_desc_sw128(sa + KPS * LW_A_BYTES + j * (sp.N * LW_BK * 2), 1024, 16);
#pragma unroll
            for (int k = 0; k < LW_BK / 16; ++k) tc_mma_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | j | k) != 0);
          }
          tc_commit(empty_bar + stage);
          if (++stage == sp.stages) { stage = 0; phase ^= 1u; }
        }
        tc_commit(tmem_full + buf);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 0-3)
    // this lane keeps the running statistics of columns `lane` and `lane + 32`
    LmColStats run[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      run[h].m = -INFINITY; run[h].s = 0.f; run[h].t = 0.f;
      run[h].v1 = -INFINITY; run[h].v2 = -INFINITY; run[h].i1 = -1; run[h].i2 = -1;
    }
    const float c = p.c;
    for (int t = 0; t < n_tiles; ++t) {
      const int buf = t & 1;
      mbar_wait(tmem_full + buf, (t >> 1) & 1u, p.dev_status);
      tc_fence_after();
      const int v_lane0 = v_begin + t * LW_BM + warp * 32;    // vocabulary entry of lane 0
      const bool valid = v_lane0 + lane < v_end;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h * 32 >= sp.N) break;
        uint32_t r[32];
        tmem_ld32(tmem_base + (static_cast<uint32_t>(warp * 32) << 16) + static_cast<uint32_t>(buf * 64 + h * 32), r);
        tc_wait_ld();
        if (h * 32 + 32 >= sp.N) {                // last chunk read: the accumulator may be overwritten
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(tmem_empty + buf);
        }
        lm_rows_chunk<kEntropy>(r, valid, v_lane0 + lane, h * 32, sp.N, lane, c, run[h]);
      }
    }
    // the four warps covered different vocabulary entries of every tile: merge through shared memory
    red[warp * 64 + lane] = run[0];
    red[warp * 64 + 32 + lane] = run[1];
    asm volatile("bar.sync 2, 128;" ::: "memory");   // the four epilogue warps
    if (warp == 0) {
      pdl_wait();   // the partials of the previous pass may still be read until earlier kernels are done
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int col = h * 32 + lane;
        if (col >= p.T) continue;
        LmColStats q = red[col];
        LmRowAcc a = {q.m, q.s, q.t};
        for (int w2 = 1; w2 < 4; ++w2) {
          const LmColStats o2 = red[w2 * 64 + col];
          lm_fold(a, o2.m, o2.s, o2.t, c);
          lm_top2_insert(o2.v1, o2.i1, q.v1, q.i1, q.v2, q.i2);
          lm_top2_insert(o2.v2, o2.i2, q.v1, q.i1, q.v2, q.i2);
        }
        LmPartial out;
        out.m = a.m; out.s = a.s; out.v1 = q.v1; out.v2 = q.v2; out.i1 = q.i1; out.i2 = q.i2; out.t = a.t; out.pad = 0;
        p.partial[static_cast<size_t>(range) * LW_ROWS + col] = out;
      }
    }
  }
  pdl_wait();
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 128);
  }
}

// One active sequence takes the W-on-M kernel (lmhead_rows_kernel): one CTA and one vocabulary range
// per SM, LW_ROWS partial rows per range.
static bool lm_rows_path(int n_seq) { return n_seq == 1; }
static thread_local int tl_lm_reserved_sms = 0;
void lm_reserve_sms_once(int n) { tl_lm_reserved_sms = n > 0 ? n : 0; }

struct LmPlan {
  int n_seq, n_mt;
  int n_ranges;    // pair kernel: vocabulary ranges of the main part; single-sequence kernel: ranges (= CTAs)
  int n_tail;      // pair kernel: pairs that sweep all M tiles over a slice of the vocabulary's tail
  int main_units;  // 32-column units of the main part
  size_t partial_rows() const { return static_cast<size_t>(n_ranges + n_tail) * n_mt * 2 * LM_BM; }
};

// `max_ws` bounds the partial array (the no-allocation entry point has a fixed one): tail pairs, which
// cost n_mt x 256 partial rows each, are given up until it fits.
static int lm_plan(const trispec_lmhead_args* a, LmPlan* pl, size_t max_ws = ~static_cast<size_t>(0)) {
  if (!a || a->B <= 0 || a->T <= 0 || a->d <= 0 || a->V <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->T > 64 || (a->d % LM_BK) != 0 || a->V < 2) return TRISPEC_ERR_UNSUPPORTED;
  pl->n_seq = a->seq_index ? a->B_active : a->B;
  if (pl->n_seq <= 0 || pl->n_seq > a->B) return TRISPEC_ERR_INVALID_ARG;
  pl->n_tail = 0;
  pl->main_units = (a->V + 31) / 32;
  if (lm_rows_path(pl->n_seq)) {
    pl->n_mt = 1;
    const int V16 = (a->V + 15) / 16;
    int sms = device_sm_count() - tl_lm_reserved_sms;
    if (sms < 1) sms = 1;
    pl->n_ranges = sms < V16 ? sms : V16;
    return TRISPEC_OK;
  }
  pl->n_mt = (pl->n_seq + 3) / 4;
  const int pairs = device_sm_count() / 2;       // one CTA pair per two SMs
  int r = pairs / pl->n_mt;
  if (r < 1) r = 1;
  const int V32 = (a->V + 31) / 32;
  if (r > V32) r = V32;
  pl->n_ranges = r;
  // Pairs that the M tiles leave over (74 = 16 x 4 + 10 for 64 sequences) take the tail of the vocabulary,
  // every one of them for all M tiles in turn. Balance in whole tiles (a tile costs a k-loop whatever its
  // width): a main pair runs ceil(main_units / r / 8) tiles, a tail pair n_mt x ceil(slice / 8).
  int tail = pairs - pl->n_mt * r;
  if (pl->n_mt < 2 || tail < 1 || pl->n_mt * r > pairs) tail = 0;
  while (tail > 0 && static_cast<size_t>(r + tail) * pl->n_mt * 2 * LM_BM * sizeof(LmPartial) > max_ws) --tail;
  if (tail > 0) {
    int best_slice = 0, best_cost = (V32 / r + 7) / 8 + 1;    // without a tail: the longest main range
    {
      const int base = V32 / r, rem = V32 - base * r;
      best_cost = (base + (rem ? ((8 - (base & 7)) < rem ? (8 - (base & 7)) : rem) : 0) + 7) / 8;
    }
    const int ideal = static_cast<int>((static_cast<long long>(V32) * tail) / (static_cast<long long>(pl->n_mt) * r + tail) / tail);
    for (int slice = (ideal / 8 > 1 ? ideal / 8 - 1 : 1) * 8; slice <= (ideal / 8 + 2) * 8; slice += 8) {
      const int main_u = V32 - slice * tail;
      if (main_u < r) break;
      const int base = main_u / r, rem = main_u - base * r;
      const int chunk = 8 - (base & 7);
      const int longest = base + (rem ? (chunk < rem ? chunk : rem) : 0);
      const int main_tiles = (longest + 7) / 8, tail_tiles = pl->n_mt * (slice / 8);
      const int cost = main_tiles > tail_tiles ? main_tiles : tail_tiles;
      if (cost < best_cost) { best_cost = cost; best_slice = slice; }
    }
    if (best_slice > 0) {
      pl->n_tail = tail;
      pl->main_units = V32 - best_slice * tail;
    }
  }
  return TRISPEC_OK;
}

}  // namespace trispec

extern "C" size_t trispec_lmhead_stats_workspace(const trispec_lmhead_args* a) {
  using namespace trispec;
  LmPlan pl;
  if (lm_plan(a, &pl) != TRISPEC_OK) return 0;
  if (lm_rows_path(pl.n_seq)) return static_cast<size_t>(pl.n_ranges) * LW_ROWS * sizeof(LmPartial);
  return pl.partial_rows() * sizeof(LmPartial);
}

namespace trispec {
static int lmhead_stats_planned(const trispec_lmhead_args* a, const LmPlan& pl, size_t ws_needed, void* stream);
}

extern "C" int trispec_lmhead_stats(const trispec_lmhead_args* a, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  LmPlan pl;
  int rc = lm_plan(a, &pl);
  const size_t ws_needed = trispec_lmhead_stats_workspace(a);
  tl_lm_reserved_sms = 0;            // a reservation holds for one call
  if (rc != TRISPEC_OK) return rc;
  return lmhead_stats_planned(a, pl, ws_needed, stream);
}

static int trispec::lmhead_stats_planned(const trispec_lmhead_args* a, const LmPlan& pl, size_t ws_needed, void* stream) {
  const int n_seq = pl.n_seq, n_mt = pl.n_mt, n_ranges = pl.n_ranges;
  int rc = TRISPEC_OK;
  if (!a->h || !a->W || !a->parent || !a->tok || !a->workspace) return TRISPEC_ERR_INVALID_ARG;
  if (!aligned16(a->h) || !aligned16(a->W) || (reinterpret_cast<uintptr_t>(a->workspace) & 255u))
    return TRISPEC_ERR_INVALID_ARG;
  if (!(a->logit_scale > 0.f) || !isfinite(a->logit_scale)) return TRISPEC_ERR_INVALID_ARG;
  const trispec_stats& o = a->out;
  if (!o.max || !o.lse || !o.top1_val || !o.top2_val || !o.p_top1 || !o.p_top2 || !o.top1_idx || !o.top2_idx ||
      !o.draft_logit || !o.p_draft)
    return TRISPEC_ERR_INVALID_ARG;
  if (a->workspace_bytes < ws_needed) return TRISPEC_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  CUtensorMap tm_h, tm_w;
  {
    const uint64_t dims[3] = {static_cast<uint64_t>(a->d), static_cast<uint64_t>(a->T), static_cast<uint64_t>(a->B)};
    const uint64_t strides[2] = {static_cast<uint64_t>(a->d) * 2, static_cast<uint64_t>(a->d) * 2 * a->T};
    const uint32_t box[3] = {LM_BK, 64, 1};
    if (!cached_tmap_bf16(&tm_h, a->h, 3, dims, strides, box)) return TRISPEC_ERR_CUDA;
  }
  {
    const uint64_t dims[2] = {static_cast<uint64_t>(a->d), static_cast<uint64_t>(a->V)};
    const uint64_t strides[1] = {static_cast<uint64_t>(a->d) * 2};
    const uint32_t box[2] = {LM_BK, 64};
    if (!cached_tmap_bf16(&tm_w, a->W, 2, dims, strides, box)) return TRISPEC_ERR_CUDA;
  }
  // the entropy sum costs two more instructions per logit: only computed when it is asked for
  const bool want_entropy = a->out.entropy != nullptr;
  LmFinalizeParams f;
  f.T = a->T; f.d = a->d; f.V = a->V; f.n_mt = n_mt; f.n_ranges = n_ranges + pl.n_tail;
  f.scale = a->logit_scale; f.c = a->logit_scale * kLog2e;
  f.seq_index = a->seq_index;
  f.partial = static_cast<LmPartial*>(a->workspace);
  f.h = static_cast<const uint16_t*>(a->h);
  f.W = static_cast<const uint16_t*>(a->W);
  f.parent = a->parent; f.tok = a->tok;
  f.out = a->out;
  if (lm_rows_path(n_seq)) {
    LmRowsParams sp;
    sp.base.T = a->T; sp.base.d = a->d; sp.base.V = a->V;
    sp.base.n_seq = 1; sp.base.n_mt = 1; sp.base.n_ranges = n_ranges;
    sp.base.n_tail = 0; sp.base.main_units = pl.main_units;
    sp.base.c = f.c;
    sp.base.seq_index = a->seq_index;
    sp.base.partial = static_cast<LmPartial*>(a->workspace);
    sp.base.dev_status = a->dev_status;
    sp.N = ((a->T + 15) / 16) * 16;
    const int kps = (a->V % 8) == 0 ? 4 : 1;
    sp.stage_bytes = kps * (LW_A_BYTES + sp.N * LW_BK * 2);
    sp.stages = (216 * 1024) / sp.stage_bytes;
    if (sp.stages > LW_MAX_STAGES) sp.stages = LW_MAX_STAGES;
    const int smem_bytes = sp.stages * sp.stage_bytes + 1024 + 8192;
    // the longer of the two range lengths (they differ by 16 rows) decides the height of the second box
    {
      const int V16 = (a->V + 15) / 16;
      const int r_big = ((V16 + n_ranges - 1) / n_ranges) * 16;
      const int last = r_big - LW_BM * ((r_big + LW_BM - 1) / LW_BM - 1);
      sp.tail_rows = last < LW_BM ? last : 0;
    }
    CUtensorMap tm_w128, tm_wt, tm_hn;
    for (int m = 0; m < 2; ++m) {
      const uint32_t rows = m == 0 ? LW_BM : static_cast<uint32_t>(sp.tail_rows);
      CUtensorMap* tm = m == 0 ? &tm_w128 : &tm_wt;
      if (rows == 0) { tm_wt = tm_w128; break; }
      if (kps == 1) {
        const uint64_t dims[2] = {static_cast<uint64_t>(a->d), static_cast<uint64_t>(a->V)};
        const uint64_t strides[1] = {static_cast<uint64_t>(a->d) * 2};
        const uint32_t box[2] = {LW_BK, rows};
        if (!cached_tmap_bf16(tm, a->W, 2, dims, strides, box)) return TRISPEC_ERR_CUDA;
      } else {
        // [V/8 groups][d/64 k-blocks][8 rows][64 elements]: the k-block index moves 128 B, the row 2 d B
        const uint64_t dims[4] = {LW_BK, 8, static_cast<uint64_t>(a->d / LW_BK), static_cast<uint64_t>(a->V / 8)};
        const uint64_t strides[3] = {static_cast<uint64_t>(a->d) * 2, LW_BK * 2, static_cast<uint64_t>(a->d) * 16};
        const uint32_t box[4] = {LW_BK, 8, static_cast<uint32_t>(kps), rows / 8};
        if (!cached_tmap_bf16(tm, a->W, 4, dims, strides, box)) return TRISPEC_ERR_CUDA;
      }
    }
    {
      const uint64_t dims[3] = {static_cast<uint64_t>(a->d), static_cast<uint64_t>(a->T), static_cast<uint64_t>(a->B)};
      const uint64_t strides[2] = {static_cast<uint64_t>(a->d) * 2, static_cast<uint64_t>(a->d) * 2 * a->T};
      const uint32_t box[3] = {LW_BK, static_cast<uint32_t>(sp.N), 1};
      if (!cached_tmap_bf16(&tm_hn, a->h, 3, dims, strides, box)) return TRISPEC_ERR_CUDA;
    }
    typedef void (*RowsKernel)(CUtensorMap, CUtensorMap, CUtensorMap, LmRowsParams);
    static const RowsKernel table[2][2] = {{lmhead_rows_kernel<false, 1>, lmhead_rows_kernel<false, 4>},
                                           {lmhead_rows_kernel<true, 1>, lmhead_rows_kernel<true, 4>}};
    const int wide = kps > 1 ? 1 : 0;
    const RowsKernel kernel = table[want_entropy ? 1 : 0][wide];
    static bool smem_set_rows[4][64] = {};
    rc = ensure_smem_limit(reinterpret_cast<const void*>(kernel), 227 * 1024, smem_set_rows[(want_entropy ? 2 : 0) + wide]);
    if (rc != TRISPEC_OK) return rc;
    TRISPEC_CUDA_OK(launch_dependent(kernel, static_cast<unsigned>(n_ranges), LW_THREADS,
                                     static_cast<size_t>(smem_bytes), st, 1, tm_w128, tm_wt, tm_hn, sp));
    count_launch();
    f.stride = LW_ROWS;
    TRISPEC_CUDA_OK(launch_dependent(lmhead_finalize_kernel, static_cast<unsigned>((a->T + 7) / 8),
                                     LM_FIN_THREADS, 0, st, 1, f, 1));
    count_launch();
    return TRISPEC_OK;
  }
  static bool smem_set[2][64] = {};
  rc = want_entropy
           ? ensure_smem_limit(reinterpret_cast<const void*>(lmhead_gemm_kernel<true>), LM_SMEM_BYTES, smem_set[1])
           : ensure_smem_limit(reinterpret_cast<const void*>(lmhead_gemm_kernel<false>), LM_SMEM_BYTES, smem_set[0]);
  if (rc != TRISPEC_OK) return rc;
  LmParams p;
  p.T = a->T; p.d = a->d; p.V = a->V;
  p.n_seq = n_seq; p.n_mt = n_mt; p.n_ranges = n_ranges;
  p.n_tail = pl.n_tail; p.main_units = pl.main_units;
  p.c = a->logit_scale * kLog2e;
  p.seq_index = a->seq_index;
  p.partial = static_cast<LmPartial*>(a->workspace);
  p.dev_status = a->dev_status;
  if (want_entropy) {
    TRISPEC_CUDA_OK(launch_dependent(lmhead_gemm_kernel<true>, static_cast<unsigned>(2 * (n_mt * n_ranges + pl.n_tail)), LM_THREADS,
                                     LM_SMEM_BYTES, st, 2, tm_h, tm_w, p));
  } else {
    TRISPEC_CUDA_OK(launch_dependent(lmhead_gemm_kernel<false>, static_cast<unsigned>(2 * (n_mt * n_ranges + pl.n_tail)), LM_THREADS,
                                     LM_SMEM_BYTES, st, 2, tm_h, tm_w, p));
  }
  count_launch();

  f.stride = n_mt * 2 * LM_BM;
  TRISPEC_CUDA_OK(launch_dependent(lmhead_finalize_kernel, static_cast<unsigned>((n_seq * a->T + 7) / 8),
                                   LM_FIN_THREADS, 0, st, 1, f, n_seq));
  count_launch();
  return TRISPEC_OK;
}

// ---------------------------------------------------------------------------------------
// No-allocation variant: the partial statistics live in an array that is part of the library
// image instead of a caller-provided workspace.
// ---------------------------------------------------------------------------------------
namespace trispec {
// Scratch shared by every call on a device. In host code this name is only a handle for the
// runtime's symbol table, not an address a kernel could use: the device address is looked up
// once per device with cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_lm_noalloc_scratch[TRISPEC_NOALLOC_SCRATCH_BYTES];

// Device address of the scratch array on the current device; looked up on the first call per
// device (with that device current) and remembered.
static int lm_noalloc_scratch(void** out) {
  static void* addr[64] = {};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRISPEC_ERR_CUDA;
  if (dev < 0 || dev >= 64) return TRISPEC_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_lm_noalloc_scratch) != cudaSuccess || !ptr) return TRISPEC_ERR_CUDA;
    addr[dev] = ptr;
  }
  *out = addr[dev];
  return TRISPEC_OK;
}
}  // namespace trispec

extern "C" int trispec_lmhead_stats_noalloc(const trispec_lmhead_args* a, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  // planned so that the partial array fits the built-in scratch (fewer tail pairs where they would not)
  LmPlan pl;
  int rc = lm_plan(a, &pl, TRISPEC_NOALLOC_SCRATCH_BYTES);
  if (rc != TRISPEC_OK) return rc;
  const size_t need = lm_rows_path(pl.n_seq) ? static_cast<size_t>(pl.n_ranges) * LW_ROWS * sizeof(LmPartial)
                                             : pl.partial_rows() * sizeof(LmPartial);
  if (need > TRISPEC_NOALLOC_SCRATCH_BYTES) return TRISPEC_ERR_TOO_LARGE;
  void* scratch = nullptr;
  rc = lm_noalloc_scratch(&scratch);
  if (rc != TRISPEC_OK) return rc;
  trispec_lmhead_args b = *a;     // same call, with the built-in array as its workspace
  b.workspace = scratch;
  b.workspace_bytes = TRISPEC_NOALLOC_SCRATCH_BYTES;
  return lmhead_stats_planned(&b, pl, need, stream);
}
