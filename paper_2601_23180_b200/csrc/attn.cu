// Verification attention (the attention of the parallel verification pass, Eq. 2 / Eq. 5):
// every draft-tree node attends to the whole committed context plus the tree keys its mask
// row allows. Split-KV: one CTA handles (sequence, KV head, M tile, KV split) and produces an
// unnormalised partial (O, m, l). With up to 8 splits the CTAs of one (sequence, KV head,
// M tile) form a thread-block cluster: each leaves its partial in its own shared memory and
// the cluster merges them through distributed shared memory, every CTA normalising and
// writing a slice of the rows - no scratch traffic and no second launch. With more splits
// (few sequences, long contexts) partials go to a caller-provided workspace and a second
// kernel merges them.
//
// GQA packing: the G = Hq / Hkv query heads that share a KV head are stacked on the M axis,
// row = node_local * G + head_in_group, so one K/V tile serves all of them. An M tile holds
// NPT = min(128 / G, 64) nodes.
//
// Per 64-key tile:  S = Q K^T  (tcgen05.mma M=128, N=64, K=128; Q is the A operand and lives
//                   in tensor memory for the whole kernel, K is the K-major B operand)
//                   online softmax in registers, one TMEM lane (row) per thread, exp2 domain,
//                   lazy rescaling of O (only when the running max grows by more than 2^8)
//                   P (bf16) -> shared memory, O += P V (V is the MN-major B operand)
// The kernel is bound by shared-memory bandwidth before anything else (TMA writes, operand
// reads of the MMAs, P), which is why Q is kept out of shared memory: per tile the MMAs read
// K, P and V only.
// Warps 0-3: softmax. Warp 4: one thread streams K and V by TMA (no multicast) through two
// independent rings (a K slot is free once S has read it, a V slot after O += P V); it
// initialises the ring barriers itself and starts loading before the CTA-wide set-up barrier.
// Warp 5: one thread issues the MMAs, polling for whichever of S(i+1) / P V(i) can go.
// A softmax thread computes and packs the exponentials of tile i before it waits for the P
// buffer to be free, so that only the 16-byte stores of P sit behind that wait.
// Two CTAs fit on one SM (~112 KB shared memory, 256 TMEM columns each). The 112 KB are either
// K ring 3 + V ring 3 + one P buffer (long tile loops: bytes in flight) or K ring 3 + V ring 2 +
// two P buffers (short loops: tile i waits for P V of tile i - 2 only).
// A sequence may carry fewer than T tree nodes (a pruned tree): rows past its count are not
// computed and M tiles past it do nothing.
#include <stdlib.h>

#include "attn_common.cuh"

namespace trispec {

// NP = number of P buffers. With one, the softmax of tile i waits for O += P V of tile i - 1 before
// it may overwrite P; with two (and a V ring of two slots instead of three, same shared memory) it
// waits for tile i - 2, which has long completed: the variant for short tile loops, which are bound
// by the S -> softmax -> P V chain of a CTA rather than by the bytes in flight.
template <bool kCluster, int NP>
__global__ void __launch_bounds__(AT_THREADS, 2)
verify_attn_split_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                         const __grid_constant__ CUtensorMap tm_kt, const __grid_constant__ CUtensorMap tm_vt,
                         const AttnParams p) {
  pdl_launch_dependents();
  // ---- which work item: the split index varies fastest, so that in cluster mode the CTAs of
  // one cluster are the splits of one (sequence, KV head, M tile) and cluster rank == split
  int idx = blockIdx.x;
  const int split = idx % p.n_splits; idx /= p.n_splits;
  const int mtile = idx % p.n_mt; idx /= p.n_mt;
  const int g = idx % p.Hkv;
  const int a = idx / p.Hkv;
  const int b = p.seq_index ? __ldg(p.seq_index + a) : a;
  // a length outside [0, capacity] (a stale or corrupt entry) is clamped and flagged: the block
  // table row and the cache are never read past their ends
  int L = __ldg(p.ctx_len + b);
  if (L < 0 || L > p.Lcap) {
    if (threadIdx.x == 0 && p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_BAD_LENGTH);
    L = max(0, min(L, p.Lcap));
  }
  // a pruned tree has fewer nodes: rows past them are not computed, M tiles past them do nothing
  const int nn = p.n_nodes ? max(0, min(p.T, __ldg(p.n_nodes + b))) : p.T;
  const int n_ctx_tiles = (L + AT_BN - 1) / AT_BN;
  // every sequence spreads its own context tiles evenly over the splits, so that the CTAs that
  // merge with each other finish together whatever the sequence's length
  const int tiles_per_split = max(1, (n_ctx_tiles + p.n_splits - 1) / p.n_splits);
  const int last_split = max(0, (n_ctx_tiles + tiles_per_split - 1) / tiles_per_split - 1);
  const int t_begin = split * tiles_per_split;
  const int t_end = min(n_ctx_tiles, t_begin + tiles_per_split);
  const bool has_tree = (split == last_split);
  const int n_tiles = (t_end - t_begin) + (has_tree ? 1 : 0);   // >= 1 unless this split is empty

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base_u32 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base_u32 - smem_u32(smem_raw));
  const bool misaligned = base_u32 - smem_u32(smem_raw) > static_cast<uint32_t>(AT_SMEM_BYTES - AT_SMEM_USED);
  if (misaligned && threadIdx.x == 0 && p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_SMEM_ALIGN);
  // a split past the end of this sequence's context has nothing to do; in cluster mode it
  // still takes part in the merge (with weight zero), so it may not leave early
  const bool idle_cta = (split > last_split) || misaligned || (mtile * p.NPT >= nn);
  if (!kCluster && idle_cta) return;           // the merge kernel skips it too

  constexpr int NV = (NP == 2) ? 2 : 3;         // V ring slots: K ring + V ring + P buffers = 112 KB either way
  uint8_t* sK = smem;                           // [AT_STAGES] K tiles
  uint8_t* sV = sK + AT_STAGES * AT_TILE_BYTES; // [NV] V tiles
  uint8_t* sP = sV + NV * AT_TILE_BYTES;        // [NP] P tiles
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + AT_STAGES * AT_KV_STAGE_BYTES + AT_P_BYTES);
  uint64_t* k_full = bars;                      // [3]  K tile landed
  uint64_t* k_empty = bars + AT_STAGES;         // [3]  S = Q K^T has consumed it
  uint64_t* v_full = bars + 2 * AT_STAGES;      // [NV] V tile landed
  uint64_t* v_empty = bars + 3 * AT_STAGES;     // [NV] O += P V has consumed it
  uint64_t* s_bar = bars + 4 * AT_STAGES;       // S ready in TMEM
  uint64_t* s_free = s_bar + 1;                 // S read into registers by the 128 softmax threads
  uint64_t* q_bar = s_bar + 2;                  // Q stored to TMEM by the 128 softmax threads
  uint64_t* o_bar = s_bar + 3;                  // [NP] O += P V of a tile using P buffer b complete (buffer free)
  uint64_t* p_bar = s_bar + 5;                  // [NP] P buffer b written by the 128 softmax threads
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_bar + 7);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* sPartO = smem;                                               // reuses the K/V ring at the end
  float2* sPartML = reinterpret_cast<float2*>(smem + AT_PART_ML_OFF);
  uint32_t tmem_base = 0;

  if (!idle_cta) {   // uniform for the whole CTA
  if (warp == 4) {
    // the loader owns the ring barriers: it signals the set-up barrier without waiting on it
    // and starts streaming while the other warps are still allocating TMEM and storing Q
    if (lane == 0) {
      for (int i = 0; i < AT_STAGES; ++i) { mbar_init(k_full + i, 1); mbar_init(k_empty + i, 1); }
      for (int i = 0; i < NV; ++i) { mbar_init(v_full + i, 1); mbar_init(v_empty + i, 1); }
      fence_mbar_init();
    }
    __syncwarp();
    asm volatile("bar.arrive 1, 192;" ::: "memory");
  } else {
    if (threadIdx.x == 0) {
      mbar_init(s_bar, 1); mbar_init(s_free, 128); mbar_init(q_bar, 128);
      for (int i = 0; i < NP; ++i) { mbar_init(o_bar + i, 1); mbar_init(p_bar + i, 128); }
      fence_mbar_init();
    }
    if (warp == 5) {
      tmem_alloc(tmem_slot, AT_TMEM_COLS);
      tmem_relinquish();
    }
    tc_fence_before();
    asm volatile("bar.sync 1, 192;" ::: "memory");
    tc_fence_after();
    tmem_base = *tmem_slot;
  }

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA loader
    if (lane == 0) {
      prefetch_tmap(&tm_k); prefetch_tmap(&tm_kt); prefetch_tmap(&tm_v); prefetch_tmap(&tm_vt);
      const int32_t* table = p.block_table + static_cast<long long>(b) * p.max_blocks_per_seq;
      auto block_id = [&](int t) -> int {      // fetched two tiles before it is used
        if (!p.paged || t >= t_end) return 0;
        int v = __ldg(table + t);
        if (v < 0 || v >= p.num_blocks) {
          if (p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_BAD_BLOCK);   // clamped, flagged
          v = 0;
        }
        return v;
      };
      auto load_tile = [&](int i, bool is_v, int blk) {
        const bool tree = has_tree && (i == n_tiles - 1);
        const int stage = is_v ? i % NV : i % AT_STAGES;
        uint64_t* full = (is_v ? v_full : k_full) + stage;
        uint8_t* dst = (is_v ? sV : sK) + stage * AT_TILE_BYTES;
        mbar_expect_tx(full, 2 * AT_BOX_BYTES);
        if (tree) {
          const CUtensorMap* tm = is_v ? &tm_vt : &tm_kt;
          tma_load_4d(dst, tm, full, 0, g, 0, b);
          tma_load_4d(dst + AT_BOX_BYTES, tm, full, 64, g, 0, b);
        } else {
          const CUtensorMap* tm = is_v ? &tm_v : &tm_k;
          const int c2 = p.paged ? 0 : (t_begin + i) * AT_BN;
          const int c3 = p.paged ? blk : b;
          tma_load_4d(dst, tm, full, 0, g, c2, c3);
          tma_load_4d(dst + AT_BOX_BYTES, tm, full, 64, g, c2, c3);
        }
      };
      int kblk0 = block_id(t_begin), kblk1 = block_id(t_begin + 1);
      int vblk0 = kblk0, vblk1 = kblk1;
      int next_k = 0, next_v = 0;
      uint32_t idle = 0;
      while (next_v < n_tiles) {
        bool progressed = false;
        if (next_k < n_tiles && mbar_test(k_empty + next_k % AT_STAGES, ((next_k / AT_STAGES) & 1u) ^ 1u)) {
          load_tile(next_k, false, kblk0);
          kblk0 = kblk1;
          kblk1 = block_id(t_begin + next_k + 2);
          ++next_k;
          progressed = true;
        }
        if (mbar_test(v_empty + next_v % NV, ((next_v / NV) & 1u) ^ 1u)) {
          load_tile(next_v, true, vblk0);
          vblk0 = vblk1;
          vblk1 = block_id(t_begin + next_v + 2);
          ++next_v;
          progressed = true;
        }
        if (progressed) {
          idle = 0;
        } else {
          __nanosleep(32);                    // leave the issue slots to the softmax warps
          if (++idle > kWaitPolls) {          // bounded: give up, flag, and let the kernel end
            if (p.dev_status) atomicExch(p.dev_status, 5);
            break;
          }
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    // S(i) may be issued once the softmax threads have read S(i-1) out of TMEM and K(i) has
    // landed; P V(i) once P(i) is in shared memory and V(i) has landed.
    if (lane == 0) {
      const uint32_t idesc_s = idesc_bf16(AT_BM, AT_BN, false, false);
      const uint32_t idesc_o = idesc_bf16(AT_BM, AT_D, false, true);
      const uint32_t sK_u = base_u32, sV_u = sK_u + AT_STAGES * AT_TILE_BYTES, sP_u = sV_u + NV * AT_TILE_BYTES;
      mbar_wait(q_bar, 0, p.dev_status);
      tc_fence_after();
      int next_s = 0, next_pv = 0;
      uint32_t idle = 0;
      while (next_pv < n_tiles) {
        bool progressed = false;
        if (next_s < n_tiles && (next_s == 0 || mbar_test(s_free, (next_s - 1) & 1u)) &&
            mbar_test(k_full + next_s % AT_STAGES, (next_s / AT_STAGES) & 1u)) {
          const int stage = next_s % AT_STAGES;
          tc_fence_after();
          const uint32_t sk = sK_u + stage * AT_TILE_BYTES;
#pragma unroll
          for (int kk = 0; kk < AT_D / 16; ++kk) {
            const uint64_t bd = smem_desc_sw128(sk + (kk >> 2) * AT_BOX_BYTES + (kk & 3) * 32, 1024, 16);
            tc_mma_ts(tmem_base + AT_TM_S, tmem_base + AT_TM_Q + kk * 8, bd, idesc_s, kk != 0);
          }
          tc_commit(s_bar);
          tc_commit(k_empty + stage);
          ++next_s;
          progressed = true;
        }
        if (next_pv < next_s && mbar_test(p_bar + next_pv % NP, (next_pv / NP) & 1u) &&
            mbar_test(v_full + next_pv % NV, (next_pv / NV) & 1u)) {
          const int stage = next_pv % NV;
          tc_fence_after();
          const uint32_t sv = sV_u + stage * AT_TILE_BYTES;
          const uint32_t sp = sP_u + (next_pv % NP) * AT_P_BYTES;
#pragma unroll
          for (int kk = 0; kk < AT_BN / 16; ++kk) {
            const uint64_t ad = smem_desc_sw128(sp + kk * 32, 1024, 16);
            // V: MN-major, 64-dim blocks 8 KB apart (LBO), 8-key groups 1 KB apart (SBO)
            const uint64_t bd = smem_desc_sw128(sv + kk * 2048, 1024, AT_BOX_BYTES);
            tc_mma_ss(tmem_base + AT_TM_O, ad, bd, idesc_o, (next_pv | kk) != 0);
          }
          tc_commit(v_empty + stage);
          tc_commit(o_bar + next_pv % NP);
          ++next_pv;
          progressed = true;
        }
        if (progressed) {
          idle = 0;
        } else {
          // (no sleep here: the sooner an MMA is issued, the sooner its K or V slot is free again)
          if (++idle > kWaitPolls) {          // bounded: give up, flag, and let the kernel end
            if (p.dev_status) atomicExch(p.dev_status, 5);
            break;
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax (warps 0-3)
    const int row = warp * 32 + lane;
    const int node = mtile * p.NPT + row / p.G;
    const bool row_valid = (row < p.NPT * p.G) && (node < nn);
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    // Q row -> TMEM (A operand of S = Q K^T): lane = row, column c = dims (2c, 2c + 1)
    {
      const int hq = g * p.G + row % p.G;
      const uint4* src = reinterpret_cast<const uint4*>(
          p.q + ((static_cast<long long>(b) * p.T + (row_valid ? node : 0)) * p.Hq + hq) * AT_D);
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t r[32];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint4 v = make_uint4(0, 0, 0, 0);
          if (row_valid) v = __ldg(src + c * 8 + j);
          r[4 * j] = v.x; r[4 * j + 1] = v.y; r[4 * j + 2] = v.z; r[4 * j + 3] = v.w;
        }
        tmem_st32(tmem_base + lane_base + AT_TM_Q + c * 32, r);
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(q_bar);
    }
    float m_ref = -INFINITY, l = 0.f;

    for (int i = 0; i < n_tiles; ++i) {
      const bool tree = has_tree && (i == n_tiles - 1);
      mbar_wait(s_bar, i & 1u, p.dev_status);
      tc_fence_after();
      uint32_t sr[64];
      {
        uint32_t r0[32], r1[32];
        tmem_ld32(tmem_base + lane_base + AT_TM_S, r0);
        tmem_ld32(tmem_base + lane_base + AT_TM_S + 32, r1);
        tc_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) { sr[j] = r0[j]; sr[32 + j] = r1[j]; }
      }
      tc_fence_before();
      mbar_arrive(s_free);                       // S(i + 1) may overwrite the buffer now
      // which keys of this tile does this row see
      uint64_t vis;
      int nvalid = AT_BN;
      if (tree) {
        // the mask comes from the kernel before this one on the stream: first dependent read
        pdl_wait();
        vis = row_valid ? __ldg(p.mask + static_cast<long long>(b) * p.T + node) : 0ull;
      } else {
        nvalid = min(AT_BN, L - (t_begin + i) * AT_BN);
        vis = (nvalid >= 64) ? ~0ull : ((1ull << nvalid) - 1ull);
      }
      // running maximum on the raw scores (the scale is positive, so it commutes with max);
      // four chains for instruction-level parallelism
      float tm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      if (!tree && nvalid >= AT_BN) {
#pragma unroll
        for (int j = 0; j < 64; j += 8) {
          tm[0] = fmax3(tm[0], __uint_as_float(sr[j]), __uint_as_float(sr[j + 1]));
          tm[1] = fmax3(tm[1], __uint_as_float(sr[j + 2]), __uint_as_float(sr[j + 3]));
          tm[2] = fmax3(tm[2], __uint_as_float(sr[j + 4]), __uint_as_float(sr[j + 5]));
          tm[3] = fmax3(tm[3], __uint_as_float(sr[j + 6]), __uint_as_float(sr[j + 7]));
        }
      } else {
#pragma unroll
        for (int j = 0; j < 64; ++j) {
          const float v = ((vis >> j) & 1ull) ? __uint_as_float(sr[j]) : -INFINITY;
          sr[j] = __float_as_uint(v);
          tm[j & 3] = fmaxf(tm[j & 3], v);
        }
      }
      const float tmax = fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3])) * p.scale_log2;
      // new reference maximum (lazy: only when the running one is exceeded by more than the
      // threshold); the rescaling of O it implies is applied further down, after P V of the
      // previous tile, so that the exponentials below do not wait for that MMA
      bool need = false;
      float f = 1.f;
      if (i == 0) {
        m_ref = tmax;
      } else {
        need = tmax > m_ref + kRescaleThreshold;
        if (need) { f = (m_ref == -INFINITY) ? 0.f : ex2f(m_ref - tmax); m_ref = tmax; l *= f; }
      }
      const float nmu = (m_ref == -INFINITY) ? 0.f : -m_ref;
      float2 ls[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
      const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nmu2 = make_float2(nmu, nmu);
      uint4 pk[8];
#pragma unroll
      for (int cch = 0; cch < 8; ++cch) {
        float e[8];
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
          // exp2(s * scale - m) on two scores at a time
          const float2 t = ffma2(make_float2(__uint_as_float(sr[cch * 8 + j]), __uint_as_float(sr[cch * 8 + j + 1])),
                                 sc2, nmu2);
          e[j] = ex2f(t.x);
          e[j + 1] = ex2f(t.y);
          ls[(j >> 1) & 1] = fadd2(ls[(j >> 1) & 1], make_float2(e[j], e[j + 1]));
        }
        pk[cch].x = pack_bf16(e[0], e[1]); pk[cch].y = pack_bf16(e[2], e[3]);
        pk[cch].z = pack_bf16(e[4], e[5]); pk[cch].w = pack_bf16(e[6], e[7]);
      }
      if (i >= NP) {
        // the P buffer is free once O += P V of the tile that used it last is complete
        mbar_wait(o_bar + i % NP, ((i / NP) - 1) & 1u, p.dev_status);
        tc_fence_after();
      }
      if (i > 0) {
        if (__any_sync(0xffffffffu, need)) {
          if (NP > 1) {   // O is stable only after the previous tile's P V
            mbar_wait(o_bar + (i - 1) % NP, ((i - 1) / NP) & 1u, p.dev_status);
            tc_fence_after();
          }
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            tmem_ld32(tmem_base + lane_base + AT_TM_O + c * 32, o);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * f);
            tmem_st32(tmem_base + lane_base + AT_TM_O + c * 32, o);
          }
          tc_wait_st();
        }
      }
      uint8_t* prow = sP + (i % NP) * AT_P_BYTES + row * 128;
#pragma unroll
      for (int cch = 0; cch < 8; ++cch) *reinterpret_cast<uint4*>(prow + ((cch ^ (row & 7)) << 4)) = pk[cch];
      l += (ls[0].x + ls[0].y) + (ls[1].x + ls[1].y);
      // keys past the end of the context, and tree nodes past the end of a pruned tree, have
      // probability 0 but their V rows may hold anything (0 * NaN = NaN): zero them
      const int vrows = tree ? ((nn < p.T) ? nn : AT_BN) : nvalid;
      if (vrows < AT_BN) {
        mbar_wait(v_full + i % NV, (i / NV) & 1u, p.dev_status);
        uint8_t* sv = sV + (i % NV) * AT_TILE_BYTES;
        for (int e = threadIdx.x; e < (AT_BN - vrows) * 16; e += 128) {
          const int r = vrows + (e >> 4), c16 = e & 15;
          *reinterpret_cast<uint4*>(sv + (c16 >> 3) * AT_BOX_BYTES + r * 128 + ((c16 & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(p_bar + i % NP);
    }
    // ---------------------------------------------------------------- epilogue
    mbar_wait(o_bar + (n_tiles - 1) % NP, ((n_tiles - 1) / NP) & 1u, p.dev_status);   // the last P V, hence all of them
    tc_fence_after();
    if (kCluster && p.n_splits == 1) {
      // a single split is the whole result: normalise and store it straight from tensor memory
      pdl_wait();                                // before the first global write
      const float invl = (l > 0.f) ? 1.f / l : 0.f;
      const int hq = g * p.G + row % p.G;
      uint16_t* orow = p.o + ((static_cast<size_t>(b) * p.T + (row_valid ? node : 0)) * p.Hq + hq) * AT_D;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t o[32];
        tmem_ld32(tmem_base + lane_base + AT_TM_O + c * 32, o);
        tc_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            uint4 pk;
            pk.x = pack_bf16(__uint_as_float(o[j]) * invl, __uint_as_float(o[j + 1]) * invl);
            pk.y = pack_bf16(__uint_as_float(o[j + 2]) * invl, __uint_as_float(o[j + 3]) * invl);
            pk.z = pack_bf16(__uint_as_float(o[j + 4]) * invl, __uint_as_float(o[j + 5]) * invl);
            pk.w = pack_bf16(__uint_as_float(o[j + 6]) * invl, __uint_as_float(o[j + 7]) * invl);
            *reinterpret_cast<uint4*>(orow + c * 32 + j) = pk;
          }
        }
      }
      if (row_valid && p.lse) p.lse[(static_cast<size_t>(b) * p.Hq + hq) * p.T + node] = (m_ref + log2f(l)) * kLn2;
    } else if (kCluster) {
      // partial (O / l as bf16, m, l) -> this CTA's shared memory (the K/V ring is idle: every
      // tile has been consumed by its MMAs). The exchange between the CTAs of a cluster goes
      // over the SM-to-SM network, whose bandwidth is a small fraction of shared memory's, so the
      // partial travels normalised and in the output precision; m and l stay fp32. Rows are
      // padded by 16 bytes so that the 16-byte stores of a warp spread over the banks.
      uint8_t* po = sPartO + row * AT_PART_PITCH;
      const float invl = (l > 0.f) ? 1.f / l : 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t o[32];
        tmem_ld32(tmem_base + lane_base + AT_TM_O + c * 32, o);
        tc_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          uint4 pk;
          pk.x = pack_bf16(__uint_as_float(o[j]) * invl, __uint_as_float(o[j + 1]) * invl);
          pk.y = pack_bf16(__uint_as_float(o[j + 2]) * invl, __uint_as_float(o[j + 3]) * invl);
          pk.z = pack_bf16(__uint_as_float(o[j + 4]) * invl, __uint_as_float(o[j + 5]) * invl);
          pk.w = pack_bf16(__uint_as_float(o[j + 6]) * invl, __uint_as_float(o[j + 7]) * invl);
          *reinterpret_cast<uint4*>(po + (c * 32 + j) * 2) = pk;
        }
      }
      sPartML[row] = make_float2(m_ref, l);
    } else {
      pdl_wait();                                // before the first global write
      const size_t item = static_cast<size_t>(blockIdx.x);
      float* po = p.part_o + (item * AT_BM + row) * AT_D;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t o[32];
        tmem_ld32(tmem_base + lane_base + AT_TM_O + c * 32, o);
        tc_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int j = 0; j < 32; j += 4)
            *reinterpret_cast<float4*>(po + c * 32 + j) =
                make_float4(__uint_as_float(o[j]), __uint_as_float(o[j + 1]), __uint_as_float(o[j + 2]),
                            __uint_as_float(o[j + 3]));
        }
      }
      if (row_valid) {
        float2 ml = make_float2(m_ref, l);
        *reinterpret_cast<float2*>(p.part_ml + (item * AT_BM + row) * 2) = ml;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem_base, AT_TMEM_COLS);
  }
  }   // !idle_cta

  if (kCluster && p.n_splits > 1) {
    // ---------------------------------------------------------------- cluster merge
    // Every CTA of the cluster holds one partial in its shared memory (idle CTAs: weight zero).
    // CTA `split` normalises rows [split * rpc, (split + 1) * rpc) of the 128.
    if (idle_cta) {
      for (int r = threadIdx.x; r < AT_BM; r += AT_THREADS) sPartML[r] = make_float2(-INFINITY, 0.f);
    }
    pdl_wait();                                  // before the first global write (o, lse)
    cluster_sync_all();
    // Requests over the SM-to-SM network are expensive per instruction, whatever their size,
    // so they are few and wide: one gather of the (m, l) pairs of all splits for this CTA's
    // rows, then per pair of rows one 16-byte-per-lane load from every split.
    // rows this CTA normalises: an even share of the 128 (the last CTA may get fewer)
    const int rpc = (((AT_BM + p.n_splits - 1) / p.n_splits) + 1) & ~1;
    const uint32_t po_u = smem_u32(sPartO), pml_u = smem_u32(sPartML);
    float2* sML2 = reinterpret_cast<float2*>(smem + AT_PART_ML2_OFF);   // [n_splits][rpc]
    for (int t = threadIdx.x; t < p.n_splits * rpc; t += AT_THREADS) {
      const int s_src = t / rpc, row = split * rpc + t % rpc;
      if (row < AT_BM) sML2[t] = ld_cluster_f2(cluster_map(pml_u + row * 8, s_src));
    }
    __syncthreads();
    constexpr int kWarps = AT_THREADS / 32;
    const int half = lane >> 4, chunk = lane & 15;
    for (int pr = warp; pr < rpc / 2; pr += kWarps) {
      const int rl = 2 * pr + half;               // row within this CTA's slice
      const int row = split * rpc + rl;
      const int node = mtile * p.NPT + row / p.G;
      const bool ok = (row < AT_BM) && (row < p.NPT * p.G) && (node < nn);
      uint4 v[8];
      float2 ml[8];
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        v[s] = make_uint4(0u, 0u, 0u, 0u);
        ml[s] = make_float2(-INFINITY, 0.f);
        if (s < p.n_splits) {
          ml[s] = sML2[s * rpc + rl];
          if (ok && ml[s].x != -INFINITY)         // an empty partial's rows hold arbitrary bits
            v[s] = ld_cluster_u4(cluster_map(po_u + row * AT_PART_PITCH + chunk * 16, s));
        }
      }
      if (!ok) continue;
      float M = -INFINITY;
#pragma unroll
      for (int s = 0; s < 8; ++s) M = fmaxf(M, ml[s].x);
      float Lsum = 0.f;
      float acc[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const float wgt = (ml[s].x != -INFINITY) ? ex2f(ml[s].x - M) * ml[s].y : 0.f;
        Lsum += wgt;
        const uint32_t w[4] = {v[s].x, v[s].y, v[s].z, v[s].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[2 * j] = fmaf(__uint_as_float(w[j] << 16), wgt, acc[2 * j]);
          acc[2 * j + 1] = fmaf(__uint_as_float(w[j] & 0xffff0000u), wgt, acc[2 * j + 1]);
        }
      }
      const float inv = 1.f / Lsum;
      const int hq = g * p.G + row % p.G;
      uint4 out;
      out.x = pack_bf16(acc[0] * inv, acc[1] * inv);
      out.y = pack_bf16(acc[2] * inv, acc[3] * inv);
      out.z = pack_bf16(acc[4] * inv, acc[5] * inv);
      out.w = pack_bf16(acc[6] * inv, acc[7] * inv);
      uint16_t* orow = p.o + ((static_cast<size_t>(b) * p.T + node) * p.Hq + hq) * AT_D;
      *reinterpret_cast<uint4*>(orow + chunk * 8) = out;
      if (p.lse && chunk == 0)
        p.lse[(static_cast<size_t>(b) * p.Hq + hq) * p.T + node] = (M + log2f(Lsum)) * kLn2;
    }
    cluster_sync_all();   // nobody leaves while its shared memory may still be read
  }
}

// ---------------------------------------------------------------------------------------
// Merge of the KV splits: one warp per output row (sequence, node, query head).
// ---------------------------------------------------------------------------------------
struct AttnMergeParams {
  int T, Hq, Hkv, G, NPT, n_mt, n_splits, n_seq, Lcap;
  const int32_t *ctx_len, *seq_index, *n_nodes;
  const float *part_o, *part_ml;
  uint16_t* o;   // bf16 [B][T][Hq][128]
  float* lse;    // [B][Hq][T] or null
};

__global__ void __launch_bounds__(256)
verify_attn_merge_kernel(const AttnMergeParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long w = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  const long long total = static_cast<long long>(p.n_seq) * p.T * p.Hq;
  if (w >= total) return;
  const int hq = static_cast<int>(w % p.Hq);
  const int node = static_cast<int>((w / p.Hq) % p.T);
  const int a = static_cast<int>(w / (static_cast<long long>(p.Hq) * p.T));
  const int b = p.seq_index ? __ldg(p.seq_index + a) : a;
  if (p.n_nodes && node >= __ldg(p.n_nodes + b)) return;   // not a node of this (pruned) tree
  const int g = hq / p.G, j = hq % p.G;
  const int mtile = node / p.NPT;
  const int row = (node % p.NPT) * p.G + j;
  const int L = max(0, min(__ldg(p.ctx_len + b), p.Lcap));   // clamped as in the split kernel
  const int n_ctx_tiles = (L + AT_BN - 1) / AT_BN;
  const int tiles_per_split = max(1, (n_ctx_tiles + p.n_splits - 1) / p.n_splits);
  const int n_valid = max(0, (n_ctx_tiles + tiles_per_split - 1) / tiles_per_split - 1) + 1;
  const size_t item0 = ((static_cast<size_t>(a) * p.Hkv + g) * p.n_mt + mtile) * p.n_splits;
  float M = -INFINITY;
  for (int s = 0; s < n_valid; ++s) {
    const size_t item = item0 + static_cast<size_t>(s);
    M = fmaxf(M, __ldg(p.part_ml + (item * AT_BM + row) * 2));
  }
  float Lsum = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < n_valid; ++s) {
    const size_t item = item0 + static_cast<size_t>(s);
    const float2 ml = __ldg(reinterpret_cast<const float2*>(p.part_ml + (item * AT_BM + row) * 2));
    const float wgt = (ml.x == -INFINITY) ? 0.f : ex2f(ml.x - M);
    Lsum += ml.y * wgt;
    const float4 v = __ldg(reinterpret_cast<const float4*>(p.part_o + (item * AT_BM + row) * AT_D) + lane);
    acc.x = fmaf(v.x, wgt, acc.x); acc.y = fmaf(v.y, wgt, acc.y);
    acc.z = fmaf(v.z, wgt, acc.z); acc.w = fmaf(v.w, wgt, acc.w);
  }
  const float inv = 1.f / Lsum;
  uint2 out;
  out.x = pack_bf16(acc.x * inv, acc.y * inv);
  out.y = pack_bf16(acc.z * inv, acc.w * inv);
  uint16_t* orow = p.o + ((static_cast<size_t>(b) * p.T + node) * p.Hq + hq) * AT_D;
  *reinterpret_cast<uint2*>(orow + lane * 4) = out;
  if (p.lse && lane == 0) p.lse[(static_cast<size_t>(b) * p.Hq + hq) * p.T + node] = (M + log2f(Lsum)) * kLn2;
}

struct AttnPlan {
  int n_seq, G, NPT, n_mt, tiles_max, n_splits;
  bool cluster;      // splits merged inside a thread-block cluster (no workspace)
  bool pieces;       // persistent CTAs over balanced pieces of the work (attn_pieces.cu)
  int n_cta;         // CTAs of the persistent launch
  size_t items;
};

// TRISPEC_ATTN_PLAN = "pieces" or "splits" overrides the planner's choice between the persistent kernel
// and the split kernels where both apply (a tuning and testing aid; read at every call).
static int attn_plan_override() {
  const char* e = getenv("TRISPEC_ATTN_PLAN");
  if (!e) return 0;
  if (e[0] == 'p') return 1;
  if (e[0] == 's') return 2;
  return 0;
}

static int attn_plan(const trispec_attn_args* a, AttnPlan* pl) {
  if (!a || a->B <= 0 || a->T <= 0 || a->Hq <= 0 || a->Hkv <= 0) return TRISPEC_ERR_INVALID_ARG;
  if (a->D != AT_D || a->T > 64 || a->Hq % a->Hkv != 0) return TRISPEC_ERR_UNSUPPORTED;
  const int G = a->Hq / a->Hkv;
  if (!(G == 1 || G == 2 || G == 4 || G == 8 || G == 16)) return TRISPEC_ERR_UNSUPPORTED;
  int Lmax;
  if (a->kv_layout == TRISPEC_KV_CONTIGUOUS) {
    if (a->Lmax < 0) return TRISPEC_ERR_INVALID_ARG;
    Lmax = a->Lmax;
  } else if (a->kv_layout == TRISPEC_KV_PAGED) {
    if (a->block_size != AT_BN) return TRISPEC_ERR_UNSUPPORTED;
    if (a->max_blocks_per_seq <= 0 || a->num_blocks <= 0) return TRISPEC_ERR_INVALID_ARG;
    Lmax = a->max_blocks_per_seq * AT_BN;
  } else {
    return TRISPEC_ERR_INVALID_ARG;
  }
  pl->n_seq = a->seq_index ? a->B_active : a->B;
  if (pl->n_seq <= 0 || pl->n_seq > a->B) return TRISPEC_ERR_INVALID_ARG;
  pl->G = G;
  pl->NPT = (AT_BM / G < 64) ? AT_BM / G : 64;
  pl->n_mt = (a->T + pl->NPT - 1) / pl->NPT;
  pl->tiles_max = (Lmax + AT_BN - 1) / AT_BN;
  const long long fixed = static_cast<long long>(pl->n_seq) * a->Hkv * pl->n_mt;
  // Number of KV splits (1..8 form a cluster; 16, 32, ... go through the workspace). Measured on the
  // five workloads: more than about 1.25 waves of CTAs with at least 32 tiles each run best (the fixed
  // costs of a CTA - pipeline fill, Q load, merge - hide behind other CTAs); when tiles are too few
  // for that, one wave filled as far as possible; very few (sequence, head) pairs are cut further.
  const long long slots = static_cast<long long>(device_sm_count()) * 2;   // two CTAs per SM (split kernels)
  const int tiles = pl->tiles_max;
  int best_s = 0;
  for (int sp = 1; sp <= 8 && !best_s; ++sp)
    if (fixed * sp * 4 >= slots * 5 && tiles / sp >= 32) best_s = sp;
  if (!best_s) {
    best_s = 1;
    for (int sp = 2; sp <= 8; ++sp)
      if (fixed * sp <= slots && tiles / sp >= 4) best_s = sp;
    if (best_s == 8 && fixed * 8 * 2 <= slots)
      for (int sp = 16; sp <= 1024 && fixed * sp <= slots && tiles / sp >= 8; sp *= 2) best_s = sp;
  }
  pl->n_splits = best_s;
  pl->cluster = pl->n_splits <= 8;
  // Clusters do not reach every CTA slot (measured: 142 of the 148 SMs take clusters of 3 or 4, 284 slots), and
  // a grid a little larger than that runs as two waves. When plain CTAs would fill the chip in ONE wave
  // (at least 92 % of all slots, long enough tile loops), that wave plus the small merge kernel is faster than
  // the clustered choice: target_escalated (96 items x 3 splits = 288 CTAs) 148 -> 118 us.
  {
    const long long cluster_slots = slots * 96 / 100;
    const int sp_full = fixed > 0 ? static_cast<int>(slots / fixed) : 0;
    if (pl->cluster && fixed * best_s > cluster_slots && sp_full >= 2 && fixed * sp_full * 100 >= slots * 92 &&
        tiles / sp_full >= 16) {
      pl->n_splits = sp_full;
      pl->cluster = false;
    }
  }
  pl->items = static_cast<size_t>(fixed) * pl->n_splits;
  if (pl->items > 0x7fffffffull) return TRISPEC_ERR_UNSUPPORTED;
  // The persistent kernel: every CTA slot of the chip gets the same number of tile steps whatever the
  // shape. It pays where the split plan cannot fill the slots evenly: fewer CTAs than slots, a last
  // wave that is mostly empty, or clusters that cannot be placed everywhere.
  pl->pieces = false;
  pl->n_cta = 0;
  if (pl->n_seq <= AT_PIECES_MAX_SEQ) {
    // groups of n_mt neighbouring CTAs (one per M tile) share a range of the (sequence, head, tile) steps
    const long long steps_max = static_cast<long long>(pl->n_seq) * a->Hkv * (tiles + 1);   // upper bound of the work
    long long n_grp = steps_max / 4;                                  // at least four steps per CTA on average
    if (n_grp > slots / pl->n_mt) n_grp = slots / pl->n_mt;
    if (n_grp < 1) n_grp = 1;
    pl->n_cta = static_cast<int>(n_grp) * pl->n_mt;
    const long long ctas = static_cast<long long>(pl->items);
    const long long waves = (ctas + slots - 1) / slots;
    const bool uneven = ctas * 100 < waves * slots * 93;              // the split plan leaves 7 % of the slots idle or more
    // The partials' trip through the workspace and the merge launch cost 15-20 us whatever the size:
    // worth it from a few hundred tile steps per CTA on (long_paged: 555 steps, 1.09 -> 0.98 ms; at 110
    // steps, llama_tree, the split plan is still ahead, 165 against 180 us).
    const int ov = attn_plan_override();
    pl->pieces = ov == 1 || (ov == 0 && uneven && steps_max >= 256 * n_grp);
  }
  return TRISPEC_OK;
}

int attn_planned_ctas(const trispec_attn_args* a) {
  AttnPlan pl;
  if (attn_plan(a, &pl) != TRISPEC_OK) return 0;
  return pl.pieces ? pl.n_cta : static_cast<int>(pl.items);
}

}  // namespace trispec

extern "C" size_t trispec_verify_attn_workspace(const trispec_attn_args* a) {
  using namespace trispec;
  AttnPlan pl;
  if (attn_plan(a, &pl) != TRISPEC_OK) return 0;
  if (pl.pieces) return attn_pieces_workspace(pl.n_cta);
  if (pl.cluster) return 0;
  return pl.items * AT_BM * (AT_D + 2) * sizeof(float);
}

extern "C" const char* trispec_verify_attn_plan(const trispec_attn_args* a) {
  using namespace trispec;
  AttnPlan pl;
  if (attn_plan(a, &pl) != TRISPEC_OK) return "none";
  return pl.pieces ? "pieces" : (pl.cluster ? "cluster" : "splits");
}

extern "C" int trispec_verify_attn(const trispec_attn_args* a, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  AttnPlan pl;
  int rc = attn_plan(a, &pl);
  if (rc != TRISPEC_OK) return rc;
  if (!a->q || !a->k_tree || !a->v_tree || !a->ctx_len || !a->mask || !a->o) return TRISPEC_ERR_INVALID_ARG;
  if ((pl.pieces || !pl.cluster) && !a->workspace) return TRISPEC_ERR_INVALID_ARG;
  if (pl.tiles_max > 0 && (!a->k_cache || !a->v_cache)) return TRISPEC_ERR_INVALID_ARG;
  if (a->kv_layout == TRISPEC_KV_PAGED && !a->block_table) return TRISPEC_ERR_INVALID_ARG;
  if (!aligned16(a->q) || !aligned16(a->k_tree) || !aligned16(a->v_tree) || !aligned16(a->k_cache) ||
      !aligned16(a->v_cache) || !aligned16(a->o) || (reinterpret_cast<uintptr_t>(a->workspace) & 255u))
    return TRISPEC_ERR_INVALID_ARG;
  if (!(a->scale > 0.f) || !isfinite(a->scale)) return TRISPEC_ERR_INVALID_ARG;
  if (a->workspace_bytes < trispec_verify_attn_workspace(a)) return TRISPEC_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  const uint64_t D = AT_D, Hkv = a->Hkv, T = a->T, B = a->B;
  CUtensorMap tm_k, tm_v, tm_kt, tm_vt;
  {
    const uint64_t dims[4] = {D, Hkv, T, B};
    const uint64_t str[3] = {D * 2, Hkv * D * 2, T * Hkv * D * 2};
    const uint32_t box[4] = {64, 1, 64, 1};
    if (!cached_tmap_bf16(&tm_kt, a->k_tree, 4, dims, str, box)) return TRISPEC_ERR_CUDA;
    if (!cached_tmap_bf16(&tm_vt, a->v_tree, 4, dims, str, box)) return TRISPEC_ERR_CUDA;
  }
  if (pl.tiles_max > 0) {
    uint64_t dims[4], str[3];
    if (a->kv_layout == TRISPEC_KV_CONTIGUOUS) {
      dims[0] = D; dims[1] = Hkv; dims[2] = a->Lmax; dims[3] = B;
      str[0] = D * 2; str[1] = Hkv * D * 2; str[2] = static_cast<uint64_t>(a->Lmax) * Hkv * D * 2;
    } else {
      dims[0] = D; dims[1] = Hkv; dims[2] = AT_BN; dims[3] = a->num_blocks;
      str[0] = D * 2; str[1] = Hkv * D * 2; str[2] = static_cast<uint64_t>(AT_BN) * Hkv * D * 2;
    }
    const uint32_t box[4] = {64, 1, 64, 1};
    if (!cached_tmap_bf16(&tm_k, a->k_cache, 4, dims, str, box)) return TRISPEC_ERR_CUDA;
    if (!cached_tmap_bf16(&tm_v, a->v_cache, 4, dims, str, box)) return TRISPEC_ERR_CUDA;
  } else {
    tm_k = tm_kt;   // never dereferenced: every sequence has zero context tiles
    tm_v = tm_vt;
  }
  // Two P buffers for CTAs with few tiles (their time is the S -> softmax -> P V chain, tile after
  // tile, and never reaches the HBM-bound steady state); one P buffer and the deeper V ring for long
  // tile loops. Measured: proxy_tree (16 tiles per CTA) 45.1 -> 43.2 us with two; long_paged
  // (128-512) 1005 -> 1023 us, target_escalated (64) 150 -> 154 us, llama_tree (129) unchanged.
  const bool two_p = pl.pieces ? (static_cast<long long>(pl.n_seq) * a->Hkv * pl.n_mt * (pl.tiles_max + 1) / pl.n_cta <= 32)
                               : (pl.tiles_max / pl.n_splits <= 32);
  typedef void (*AttnKernel)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, AttnParams);
  const AttnKernel kernel = pl.cluster ? (two_p ? verify_attn_split_kernel<true, 2> : verify_attn_split_kernel<true, 1>)
                                       : (two_p ? verify_attn_split_kernel<false, 2> : verify_attn_split_kernel<false, 1>);
  static bool smem_set[4][64] = {};
  rc = ensure_smem_limit(reinterpret_cast<const void*>(kernel), AT_SMEM_BYTES, smem_set[(pl.cluster ? 2 : 0) + (two_p ? 1 : 0)]);
  if (rc != TRISPEC_OK) return rc;
  AttnParams p;
  p.T = a->T; p.Hq = a->Hq; p.Hkv = a->Hkv; p.G = pl.G; p.NPT = pl.NPT; p.n_mt = pl.n_mt;
  p.n_splits = pl.n_splits;
  p.paged = (a->kv_layout == TRISPEC_KV_PAGED); p.max_blocks_per_seq = a->max_blocks_per_seq;
  p.num_blocks = a->num_blocks;
  p.Lcap = p.paged ? a->max_blocks_per_seq * AT_BN : a->Lmax;
  p.scale_log2 = a->scale * kLog2e;
  p.q = static_cast<const uint16_t*>(a->q);
  p.block_table = a->block_table; p.ctx_len = a->ctx_len; p.seq_index = a->seq_index; p.mask = a->mask;
  p.n_nodes = a->n_nodes;
  p.part_o = static_cast<float*>(a->workspace);
  p.part_ml = p.part_o + pl.items * AT_BM * AT_D;
  p.o = static_cast<uint16_t*>(a->o);
  p.lse = a->lse;
  p.dev_status = a->dev_status;
  p.n_seq = pl.n_seq;
  p.n_cta = pl.n_cta;
  if (pl.pieces) {
    const CUtensorMap maps[4] = {tm_k, tm_v, tm_kt, tm_vt};
    return attn_launch_pieces(p, maps, two_p, a->workspace, st);
  }
  if (pl.cluster) {
    TRISPEC_CUDA_OK(launch_dependent(kernel, static_cast<unsigned>(pl.items), AT_THREADS,
                                     AT_SMEM_BYTES, st, static_cast<unsigned>(pl.n_splits), tm_k, tm_v, tm_kt, tm_vt,
                                     p));
    count_launch();
    return TRISPEC_OK;
  }
  TRISPEC_CUDA_OK(launch_dependent(kernel, static_cast<unsigned>(pl.items), AT_THREADS,
                                   AT_SMEM_BYTES, st, 1, tm_k, tm_v, tm_kt, tm_vt, p));
  count_launch();

  AttnMergeParams m;
  m.T = a->T; m.Hq = a->Hq; m.Hkv = a->Hkv; m.G = pl.G; m.NPT = pl.NPT; m.n_mt = pl.n_mt;
  m.n_splits = pl.n_splits; m.n_seq = pl.n_seq; m.Lcap = p.Lcap;
  m.ctx_len = a->ctx_len; m.seq_index = a->seq_index; m.n_nodes = a->n_nodes;
  m.part_o = p.part_o; m.part_ml = p.part_ml;
  m.o = static_cast<uint16_t*>(a->o); m.lse = a->lse;
  const long long rows = static_cast<long long>(pl.n_seq) * a->T * a->Hq;
  TRISPEC_CUDA_OK(launch_dependent(verify_attn_merge_kernel, static_cast<unsigned>((rows + 7) / 8), 256, 0, st, 1, m));
  count_launch();
  return TRISPEC_OK;
}
