// Verification attention (Eq. 2 / Eq. 5), persistent form: a fixed number of CTAs, two per SM,
// share the work of a launch evenly whatever the number of sequences, heads and context lengths.
//
// The work of a launch is a sequence of 64-key tile steps: for every active sequence and KV head, the
// context tiles of the sequence followed by its tree tile. The CTAs form groups of n_mt neighbours, one
// CTA per M tile (128 stacked query rows; n_mt = 1 up to two query heads per KV head); group r of R
// takes the steps [r W / R, (r + 1) W / R) of that sequence of W steps, all its CTAs at the same time,
// so that a K/V tile is fetched from HBM once and found in L2 by the other M tiles. A range is cut into
// PIECES: a run of consecutive tiles of one (sequence, KV head). A CTA works through its
// pieces one after the other with the same pipeline as the split kernel (attn.cu: Q in tensor
// memory, K/V rings filled by TMA, S = Q K^T and O += P V on tcgen05, one softmax thread per row);
// the rings and their barriers run on across pieces, so the loader is already streaming the next
// piece while the softmax threads finish the current one. A piece that covers a whole
// (sequence, head, M tile) is normalised and stored directly; any other piece leaves an fp32 partial
// (O, m, l) in the caller's workspace (a CTA has at most two of those, its first and its last piece),
// and a second kernel merges the partials of the items that were cut. No CTA waits for another one.
//
// Nothing here depends on how the tile counts divide the chip: there is no wave of CTAs that ends
// early or late, and every SM hosts the same two CTAs from start to end. The price is the partials'
// trip through the workspace (L2-resident) and the second launch.
//
// The partition is computed on the device from ctx_len / n_nodes by every warp that needs it
// (a warp scan over at most 128 sequences held four per lane), identically in both kernels.
#include "attn_common.cuh"

namespace trispec {

constexpr int AP_MAX_SEQ = 128;                 // four sequences per lane

// Per-warp view of the work: for the sequences lane, lane + 32, lane + 64, lane + 96 (in the order
// of the active list) the clamped context length, the node count, the number of tile steps and
// the exclusive prefix sum of the steps over all sequences before it.
struct WorkMap {
  int L[4], nn[4], steps[4], pre[4];
  int total;
};

// steps of one sequence: KV heads x (context tiles + the tree tile); a sequence without nodes has none
__device__ __forceinline__ int seq_steps(const AttnParams& p, int L, int nn) {
  return nn > 0 ? p.Hkv * ((L + AT_BN - 1) / AT_BN + 1) : 0;
}

// warp-collective; flags out-of-range lengths like the split kernel does
__device__ __forceinline__ WorkMap load_work_map(const AttnParams& p, int lane, bool flag_bad) {
  WorkMap w;
  int run = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int a = j * 32 + lane;
    int L = 0, nn = 0;
    if (a < p.n_seq) {
      const int b = p.seq_index ? __ldg(p.seq_index + a) : a;
      L = __ldg(p.ctx_len + b);
      if (L < 0 || L > p.Lcap) {
        if (flag_bad && p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_BAD_LENGTH);
        L = max(0, min(L, p.Lcap));
      }
      nn = p.n_nodes ? max(0, min(p.T, __ldg(p.n_nodes + b))) : p.T;
    }
    w.L[j] = L;
    w.nn[j] = nn;
    w.steps[j] = (a < p.n_seq) ? seq_steps(p, L, nn) : 0;
    int incl = w.steps[j];
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    w.pre[j] = run + incl - w.steps[j];
    run += __shfl_sync(0xffffffffu, incl, 31);
  }
  w.total = run;
  return w;
}

// A run of consecutive tiles of one (sequence, KV head).
struct Piece {
  int a, g;             // position in the active list, KV head
  int L, nn;            // clamped context length and node count of the sequence
  int n_it;             // tile steps of the whole item: context tiles + 1
  int t0, t1;           // this piece's steps [t0, t1) of the item
  long long start;      // global step index of t0
};

// warp-collective: the piece that starts at global step `cur` and ends at the item's end or at `limit`
__device__ __forceinline__ Piece piece_at(const AttnParams& p, const WorkMap& w, long long cur, long long limit,
                                          int lane) {
  int a = 0, L = 0, nn = 0, pre = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const bool mine = w.steps[j] > 0 && cur >= w.pre[j] && cur < static_cast<long long>(w.pre[j]) + w.steps[j];
    const unsigned m = __ballot_sync(0xffffffffu, mine);
    if (m) {
      const int src = __ffs(m) - 1;
      a = j * 32 + src;
      L = __shfl_sync(0xffffffffu, w.L[j], src);
      nn = __shfl_sync(0xffffffffu, w.nn[j], src);
      pre = __shfl_sync(0xffffffffu, w.pre[j], src);
    }
  }
  Piece pc;
  pc.a = a; pc.L = L; pc.nn = nn;
  pc.n_it = (L + AT_BN - 1) / AT_BN + 1;
  const int local = static_cast<int>(cur - pre);
  pc.g = local / pc.n_it;
  pc.t0 = local % pc.n_it;
  pc.t1 = static_cast<int>(min(static_cast<long long>(pc.n_it), pc.t0 + (limit - cur)));
  pc.start = cur;
  return pc;
}

// warp-collective: the next piece at or after `cur` (which is advanced past it) whose sequence has nodes in
// M tile `mtile`; false when the range [cur, limit) holds no more
__device__ __forceinline__ bool next_piece(const AttnParams& p, const WorkMap& w, long long& cur, long long limit,
                                           int lane, int mtile, Piece& out) {
  while (cur < limit) {
    out = piece_at(p, w, cur, limit, lane);
    cur += out.t1 - out.t0;
    if (mtile * p.NPT < out.nn) return true;     // (a pruned tree may have no node in this M tile)
  }
  return false;
}

// first global step of group r of R, and the group that owns global step s
__device__ __forceinline__ long long cta_first_step(long long W, int C, int c) { return (W * c) / C; }
__device__ __forceinline__ int cta_of_step(long long W, int C, long long s) {
  const long long c = ((s + 1) * C + W - 1) / W - 1;
  return static_cast<int>(min(static_cast<long long>(C - 1), max(0ll, c)));
}

// NP = number of P buffers (see attn.cu): one with a V ring of three slots, two with a V ring of two.
template <int NP>
__global__ void __launch_bounds__(AT_THREADS, 2)
verify_attn_pieces_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                          const __grid_constant__ CUtensorMap tm_kt, const __grid_constant__ CUtensorMap tm_vt,
                          const AttnParams p) {
  pdl_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // The loader and the issuer warp each keep a copy of the work map (registers) and walk this CTA's
  // pieces with it; the softmax warps get every piece from the issuer through a two-entry mailbox in
  // shared memory, which keeps the map out of their registers. (All warps build the map once: whether
  // the CTA has work at all decides how it leaves.)
  const WorkMap wm = load_work_map(p, lane, warp == 4);
  const long long W = wm.total;
  const int cta = blockIdx.x;
  const int n_grp = p.n_cta / p.n_mt, grp = cta / p.n_mt, mtile = cta % p.n_mt;   // neighbours share K/V tiles
  const long long w_begin = cta_first_step(W, n_grp, grp), w_end = cta_first_step(W, n_grp, grp + 1);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base_u32 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base_u32 - smem_u32(smem_raw));
  const bool misaligned = base_u32 - smem_u32(smem_raw) > static_cast<uint32_t>(AT_SMEM_BYTES - AT_SMEM_USED);
  if (misaligned && threadIdx.x == 0 && p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_SMEM_ALIGN);
  if (w_begin >= w_end || misaligned) return;    // nothing to do (fewer steps than CTAs): the merge kernel knows

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
  uint64_t* q_bar = s_bar + 2;                  // Q of the next piece stored (and O of the last one read out)
  uint64_t* o_bar = s_bar + 3;                  // [NP] O += P V of a tile using P buffer b complete (buffer free)
  uint64_t* p_bar = s_bar + 5;                  // [NP] P buffer b written by the 128 softmax threads
  uint64_t* pc_bar = s_bar + 7;                 // the issuer has left the next piece in the mailbox
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_bar + 8);
  int* mailbox = reinterpret_cast<int*>(s_bar + 10);  // (16-byte aligned) [2][8]: a, g, L, nn, n_it, t0, t1 (t1 = t0: no more pieces), first
  uint32_t tmem_base = 0;
  auto post_piece = [&](int k, bool have, const Piece& pc) {
    int* m = mailbox + (k & 1) * 8;
    m[0] = pc.a; m[1] = pc.g; m[2] = pc.L; m[3] = pc.nn; m[4] = pc.n_it; m[5] = pc.t0;
    m[6] = have ? pc.t1 : pc.t0;
    m[7] = (pc.start == w_begin) ? 1 : 0;
  };
  // the issuer warp's walk over the pieces (used by warp 5 only)
  long long walk = w_begin;
  Piece cur_pc;
  bool have_pc = false;

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
      mbar_init(s_bar, 1); mbar_init(s_free, 128); mbar_init(q_bar, 128); mbar_init(pc_bar, 1);
      for (int i = 0; i < NP; ++i) { mbar_init(o_bar + i, 1); mbar_init(p_bar + i, 128); }
      fence_mbar_init();
    }
    if (warp == 5) {
      tmem_alloc(tmem_slot, AT_TMEM_COLS);
      tmem_relinquish();
      have_pc = next_piece(p, wm, walk, w_end, lane, mtile, cur_pc);
      if (lane == 0) post_piece(0, have_pc, cur_pc);      // the first piece: visible after the set-up barrier
    }
    tc_fence_before();
    asm volatile("bar.sync 1, 192;" ::: "memory");
    tc_fence_after();
    tmem_base = *tmem_slot;
  }

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA loader
    if (lane == 0) { prefetch_tmap(&tm_k); prefetch_tmap(&tm_kt); prefetch_tmap(&tm_v); prefetch_tmap(&tm_vt); }
    int n0 = 0;                                  // tiles of earlier pieces: the rings run on across pieces
    bool alive = true;
    for (long long cur = w_begin; cur < w_end;) {
      const Piece pc = piece_at(p, wm, cur, w_end, lane);
      const int nt = pc.t1 - pc.t0;
      if (mtile * p.NPT >= pc.nn) { cur += nt; continue; }   // a pruned tree without nodes in this M tile
      if (lane == 0 && alive) {
        const int b = p.seq_index ? __ldg(p.seq_index + pc.a) : pc.a;
        const int n_ctx = pc.n_it - 1;           // context tiles of the item; step n_ctx is the tree tile
        const int32_t* table = p.block_table + static_cast<long long>(b) * p.max_blocks_per_seq;
        auto block_id = [&](int t) -> int {      // fetched two tiles before it is used
          if (!p.paged || t >= n_ctx || t >= pc.t1) return 0;
          int v = __ldg(table + t);
          if (v < 0 || v >= p.num_blocks) {
            if (p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_BAD_BLOCK);   // clamped, flagged
            v = 0;
          }
          return v;
        };
        auto load_tile = [&](int i, bool is_v, int blk) {
          const int t = pc.t0 + i;
          const int n = n0 + i;
          const int stage = is_v ? n % NV : n % AT_STAGES;
          uint64_t* full = (is_v ? v_full : k_full) + stage;
          uint8_t* dst = (is_v ? sV : sK) + stage * AT_TILE_BYTES;
          mbar_expect_tx(full, 2 * AT_BOX_BYTES);
          if (t == n_ctx) {
            const CUtensorMap* tm = is_v ? &tm_vt : &tm_kt;
            tma_load_4d(dst, tm, full, 0, pc.g, 0, b);
            tma_load_4d(dst + AT_BOX_BYTES, tm, full, 64, pc.g, 0, b);
          } else {
            const CUtensorMap* tm = is_v ? &tm_v : &tm_k;
            const int c2 = p.paged ? 0 : t * AT_BN;
            const int c3 = p.paged ? blk : b;
            tma_load_4d(dst, tm, full, 0, pc.g, c2, c3);
            tma_load_4d(dst + AT_BOX_BYTES, tm, full, 64, pc.g, c2, c3);
          }
        };
        int kblk0 = block_id(pc.t0), kblk1 = block_id(pc.t0 + 1);
        int vblk0 = kblk0, vblk1 = kblk1;
        int next_k = 0, next_v = 0;
        uint32_t idle = 0;
        while (next_v < nt) {
          bool progressed = false;
          const int nk = n0 + next_k, nv = n0 + next_v;
          if (next_k < nt && mbar_test(k_empty + nk % AT_STAGES, ((nk / AT_STAGES) & 1u) ^ 1u)) {
            load_tile(next_k, false, kblk0);
            kblk0 = kblk1;
            kblk1 = block_id(pc.t0 + next_k + 2);
            ++next_k;
            progressed = true;
          }
          if (mbar_test(v_empty + nv % NV, ((nv / NV) & 1u) ^ 1u)) {
            load_tile(next_v, true, vblk0);
            vblk0 = vblk1;
            vblk1 = block_id(pc.t0 + next_v + 2);
            ++next_v;
            progressed = true;
          }
          if (progressed) {
            idle = 0;
          } else {
            __nanosleep(32);                    // leave the issue slots to the softmax warps
            if (++idle > kWaitPolls) {          // bounded: give up, flag, and let the kernel end
              if (p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_DEVICE_TIMEOUT);
              alive = false;
              break;
            }
          }
        }
      }
      n0 += nt;
      cur += nt;
      __syncwarp();
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    // S(n) may be issued once the softmax threads have read S(n - 1) out of TMEM and K(n) has landed;
    // P V(n) once P(n) is in shared memory and V(n) has landed. n counts the tiles of all pieces of
    // this CTA; a piece starts once its Q is in tensor memory, which also tells that the accumulator
    // of the piece before has been read out.
    const uint32_t idesc_s = idesc_bf16(AT_BM, AT_BN, false, false);
    const uint32_t idesc_o = idesc_bf16(AT_BM, AT_D, false, true);
    const uint32_t sK_u = base_u32, sV_u = sK_u + AT_STAGES * AT_TILE_BYTES, sP_u = sV_u + NV * AT_TILE_BYTES;
    int n0 = 0, piece_idx = 0;
    bool alive = true;
    while (have_pc) {
      const Piece pc = cur_pc;
      const int nt = pc.t1 - pc.t0;
      Piece nx;
      const bool have_nx = next_piece(p, wm, walk, w_end, lane, mtile, nx);
      if (lane == 0) {
        if (alive) alive = mbar_wait(q_bar, piece_idx & 1u, p.dev_status);
        // every softmax thread has taken this piece out of the mailbox, hence is done with the other entry
        post_piece(piece_idx + 1, have_nx, nx);
        mbar_arrive(pc_bar);
      }
      if (lane == 0 && alive) {
        tc_fence_after();
        int next_s = 0, next_pv = 0;
        uint32_t idle = 0;
        while (alive && next_pv < nt) {
          bool progressed = false;
          const int ns = n0 + next_s, np = n0 + next_pv;
          if (next_s < nt && (ns == 0 || mbar_test(s_free, (ns - 1) & 1u)) &&
              mbar_test(k_full + ns % AT_STAGES, (ns / AT_STAGES) & 1u)) {
            const int stage = ns % AT_STAGES;
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
          if (next_pv < next_s && mbar_test(p_bar + np % NP, (np / NP) & 1u) &&
              mbar_test(v_full + np % NV, (np / NV) & 1u)) {
            const int stage = np % NV;
            tc_fence_after();
            const uint32_t sv = sV_u + stage * AT_TILE_BYTES;
            const uint32_t sp = sP_u + (np % NP) * AT_P_BYTES;
#pragma unroll
            for (int kk = 0; kk < AT_BN / 16; ++kk) {
              const uint64_t ad = smem_desc_sw128(sp + kk * 32, 1024, 16);
              // V: MN-major, 64-dim blocks 8 KB apart (LBO), 8-key groups 1 KB apart (SBO)
              const uint64_t bd = smem_desc_sw128(sv + kk * 2048, 1024, AT_BOX_BYTES);
              tc_mma_ss(tmem_base + AT_TM_O, ad, bd, idesc_o, (next_pv | kk) != 0);
            }
            tc_commit(v_empty + stage);
            tc_commit(o_bar + np % NP);
            ++next_pv;
            progressed = true;
          }
          if (progressed) {
            idle = 0;
          } else if (++idle > kWaitPolls) {     // bounded: give up, flag, and let the kernel end
            if (p.dev_status) atomicExch(p.dev_status, TRISPEC_ERR_DEVICE_TIMEOUT);
            alive = false;
          }
        }
      }
      n0 += nt;
      cur_pc = nx;
      have_pc = have_nx;
      ++piece_idx;
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------------ softmax (warps 0-3)
    const int row = warp * 32 + lane;
    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    int n0 = 0;
    for (int piece_idx = 0;; ++piece_idx) {
      // this piece, from the issuer's mailbox
      if (piece_idx > 0 && !mbar_wait(pc_bar, (piece_idx - 1) & 1u, p.dev_status)) break;
      Piece pc;
      bool first_piece;
      {
        const int4* m = reinterpret_cast<const int4*>(mailbox + (piece_idx & 1) * 8);
        const int4 lo = m[0], hi = m[1];
        pc.a = lo.x; pc.g = lo.y; pc.L = lo.z; pc.nn = lo.w;
        pc.n_it = hi.x; pc.t0 = hi.y; pc.t1 = hi.z;
        first_piece = hi.w != 0;
      }
      const int nt = pc.t1 - pc.t0;
      if (nt <= 0) break;                          // no more pieces
      const int n_ctx = pc.n_it - 1;
      const int b = p.seq_index ? __ldg(p.seq_index + pc.a) : pc.a;
      const int node = mtile * p.NPT + row / p.G;
      const bool row_valid = (row < p.NPT * p.G) && (node < pc.nn);
      const int hq = pc.g * p.G + row % p.G;
      // Q row -> TMEM (A operand of S = Q K^T): lane = row, column c = dims (2c, 2c + 1). The S MMAs
      // of the piece before have completed (this thread saw their last result), and this thread has
      // read its accumulator row out: the issuer starts the piece once all 128 threads are here.
      {
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

      for (int i = 0; i < nt; ++i) {
        const int n = n0 + i, t = pc.t0 + i;
        const bool tree = (t == n_ctx);
        mbar_wait(s_bar, n & 1u, p.dev_status);
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
        mbar_arrive(s_free);                       // S(n + 1) may overwrite the buffer now
        // which keys of this tile does this row see
        uint64_t vis;
        int nvalid = AT_BN;
        if (tree) {
          // the mask comes from the kernel before this one on the stream: first dependent read
          pdl_wait();
          vis = row_valid ? __ldg(p.mask + static_cast<long long>(b) * p.T + node) : 0ull;
        } else {
          nvalid = min(AT_BN, pc.L - t * AT_BN);
          vis = (nvalid >= 64) ? ~0ull : ((1ull << nvalid) - 1ull);
        }
        // running maximum on the raw scores (the scale is positive, so it commutes with max)
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
            const float2 tt = ffma2(make_float2(__uint_as_float(sr[cch * 8 + j]), __uint_as_float(sr[cch * 8 + j + 1])),
                                    sc2, nmu2);
            e[j] = ex2f(tt.x);
            e[j + 1] = ex2f(tt.y);
            ls[(j >> 1) & 1] = fadd2(ls[(j >> 1) & 1], make_float2(e[j], e[j + 1]));
          }
          pk[cch].x = pack_bf16(e[0], e[1]); pk[cch].y = pack_bf16(e[2], e[3]);
          pk[cch].z = pack_bf16(e[4], e[5]); pk[cch].w = pack_bf16(e[6], e[7]);
        }
        if (n >= NP) {
          // the P buffer is free once O += P V of the tile that used it last is complete
          mbar_wait(o_bar + n % NP, ((n / NP) - 1) & 1u, p.dev_status);
          tc_fence_after();
        }
        if (i > 0) {
          if (__any_sync(0xffffffffu, need)) {
            if (NP > 1) {   // O is stable only after the previous tile's P V
              mbar_wait(o_bar + (n - 1) % NP, ((n - 1) / NP) & 1u, p.dev_status);
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
        uint8_t* prow = sP + (n % NP) * AT_P_BYTES + row * 128;
#pragma unroll
        for (int cch = 0; cch < 8; ++cch) *reinterpret_cast<uint4*>(prow + ((cch ^ (row & 7)) << 4)) = pk[cch];
        l += (ls[0].x + ls[0].y) + (ls[1].x + ls[1].y);
        // keys past the end of the context, and tree nodes past the end of a pruned tree, have
        // probability 0 but their V rows may hold anything (0 * NaN = NaN): zero them
        const int vrows = tree ? ((pc.nn < p.T) ? pc.nn : AT_BN) : nvalid;
        if (vrows < AT_BN) {
          mbar_wait(v_full + n % NV, (n / NV) & 1u, p.dev_status);
          uint8_t* sv = sV + (n % NV) * AT_TILE_BYTES;
          for (int e = threadIdx.x; e < (AT_BN - vrows) * 16; e += 128) {
            const int r = vrows + (e >> 4), c16 = e & 15;
            *reinterpret_cast<uint4*>(sv + (c16 >> 3) * AT_BOX_BYTES + r * 128 + ((c16 & 7) << 4)) = make_uint4(0, 0, 0, 0);
          }
        }
        fence_async_smem();
        tc_fence_before();
        mbar_arrive(p_bar + n % NP);
      }
      // ---------------------------------------------------------------- end of the piece
      {
        const int n_last = n0 + nt - 1;
        mbar_wait(o_bar + n_last % NP, (n_last / NP) & 1u, p.dev_status);   // the last P V, hence all of them
        tc_fence_after();
        pdl_wait();                                // before the first global write
        if (pc.t0 == 0 && pc.t1 == pc.n_it) {
          // all tiles of the (sequence, head): normalise and store the M tile straight from tensor memory
          const float invl = (l > 0.f) ? 1.f / l : 0.f;
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
        } else {
          // a part of it: unnormalised fp32 partial; slot 2c for the piece this CTA starts with, 2c + 1 for
          // the one it ends with (the pieces in between are whole)
          const size_t slot = 2 * static_cast<size_t>(cta) + (first_piece ? 0 : 1);
          float* po = p.part_o + (slot * AT_BM + row) * AT_D;
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
          if (row_valid) *reinterpret_cast<float2*>(p.part_ml + (slot * AT_BM + row) * 2) = make_float2(m_ref, l);
        }
      }
      n0 += nt;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem_base, AT_TMEM_COLS);
  }
}

// ---------------------------------------------------------------------------------------
// Merge of the partials: four blocks per (sequence, KV head, M tile), each with sixteen warps that take
// a quarter of the item's rows in turn. Every warp rebuilds the partition (before it waits for the first kernel) and
// finds the groups that shared the item; an item that was a single piece has been written by the
// first kernel and costs its block nothing more. A row's partials are folded in one pass, four
// partials' loads in flight at a time.
// ---------------------------------------------------------------------------------------
constexpr int AP_MERGE_THREADS = 512;
constexpr int AP_MERGE_BLOCKS = 4;              // blocks per item, 32 rows each

__global__ void __launch_bounds__(AP_MERGE_THREADS)
verify_attn_pieces_merge_kernel(const AttnParams p) {
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int item = blockIdx.x / AP_MERGE_BLOCKS, quarter = blockIdx.x % AP_MERGE_BLOCKS;
  const int mtile = item % p.n_mt;
  const int g = (item / p.n_mt) % p.Hkv;
  const int a = item / (p.n_mt * p.Hkv);
  const WorkMap wm = load_work_map(p, lane, false);
  // the sequence's entry of the map lives in lane a % 32, slot a / 32
  int L = 0, nn = 0, pre = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int Lj = __shfl_sync(0xffffffffu, wm.L[j], a & 31), nj = __shfl_sync(0xffffffffu, wm.nn[j], a & 31);
    const int pj = __shfl_sync(0xffffffffu, wm.pre[j], a & 31);
    if (j == (a >> 5)) { L = Lj; nn = nj; pre = pj; }
  }
  if (mtile * p.NPT >= nn) return;               // no node of this (pruned) tree in the M tile
  const int n_it = (L + AT_BN - 1) / AT_BN + 1;
  const long long W = wm.total;
  const int n_grp = p.n_cta / p.n_mt;
  const long long x = pre + static_cast<long long>(g) * n_it;                 // first global step of the (sequence, head)
  const int r_first = cta_of_step(W, n_grp, x), r_last = cta_of_step(W, n_grp, x + n_it - 1);
  if (r_first == r_last) return;                 // one piece: stored by the first kernel
  const int b = p.seq_index ? __ldg(p.seq_index + a) : a;
  pdl_wait();                                    // the partials come from the kernel before
  const int n_rows = min(min(AT_BM, p.NPT * p.G), (quarter + 1) * (AT_BM / AP_MERGE_BLOCKS));
  for (int row = quarter * (AT_BM / AP_MERGE_BLOCKS) + warp; row < n_rows; row += AP_MERGE_THREADS / 32) {
    const int node = mtile * p.NPT + row / p.G;
    if (node >= nn) break;                       // rows are in node order
    const int hq = g * p.G + row % p.G;
    float M = -INFINITY, Lsum = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r0 = r_first; r0 <= r_last; r0 += 4) {
      float2 ml[4];
      float4 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        ml[k] = make_float2(-INFINITY, 0.f);
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        const int r = r0 + k;
        if (r <= r_last) {
          // slot 2c for the piece a CTA starts with (the item began before the group's range), else 2c + 1
          const size_t c = static_cast<size_t>(r) * p.n_mt + mtile;
          const size_t slot = 2 * c + (cta_first_step(W, n_grp, r) >= x ? 0 : 1);
          ml[k] = __ldg(reinterpret_cast<const float2*>(p.part_ml + (slot * AT_BM + row) * 2));
          v[k] = __ldg(reinterpret_cast<const float4*>(p.part_o + (slot * AT_BM + row) * AT_D) + lane);
        }
      }
      float Mn = M;
#pragma unroll
      for (int k = 0; k < 4; ++k) Mn = fmaxf(Mn, ml[k].x);
      const float keep = (M == -INFINITY) ? 0.f : ex2f(M - Mn);
      Lsum *= keep;
      acc.x *= keep; acc.y *= keep; acc.z *= keep; acc.w *= keep;
      M = Mn;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float wgt = (ml[k].x == -INFINITY) ? 0.f : ex2f(ml[k].x - M);
        Lsum += ml[k].y * wgt;
        acc.x = fmaf(v[k].x, wgt, acc.x); acc.y = fmaf(v[k].y, wgt, acc.y);
        acc.z = fmaf(v[k].z, wgt, acc.z); acc.w = fmaf(v[k].w, wgt, acc.w);
      }
    }
    const float inv = (Lsum > 0.f) ? 1.f / Lsum : 0.f;
    uint2 out;
    out.x = pack_bf16(acc.x * inv, acc.y * inv);
    out.y = pack_bf16(acc.z * inv, acc.w * inv);
    uint16_t* orow = p.o + ((static_cast<size_t>(b) * p.T + node) * p.Hq + hq) * AT_D;
    *reinterpret_cast<uint2*>(orow + lane * 4) = out;
    if (p.lse && lane == 0) p.lse[(static_cast<size_t>(b) * p.Hq + hq) * p.T + node] = (M + log2f(Lsum)) * kLn2;
  }
}

size_t attn_pieces_workspace(int n_cta) {
  return static_cast<size_t>(2) * n_cta * AT_BM * (AT_D + 2) * sizeof(float);
}

// Launches the persistent kernel and its merge. `p` carries everything but the partial pointers.
int attn_launch_pieces(AttnParams p, const CUtensorMap* maps, bool two_p, void* workspace, cudaStream_t st) {
  typedef void (*Kernel)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, AttnParams);
  const Kernel kernel = two_p ? verify_attn_pieces_kernel<2> : verify_attn_pieces_kernel<1>;
  static bool smem_set[2][64] = {};
  int rc = ensure_smem_limit(reinterpret_cast<const void*>(kernel), AT_SMEM_BYTES, smem_set[two_p ? 1 : 0]);
  if (rc != TRISPEC_OK) return rc;
  p.part_o = static_cast<float*>(workspace);
  p.part_ml = p.part_o + static_cast<size_t>(2) * p.n_cta * AT_BM * AT_D;
  TRISPEC_CUDA_OK(launch_dependent(kernel, static_cast<unsigned>(p.n_cta), AT_THREADS, AT_SMEM_BYTES, st, 1, maps[0],
                                   maps[1], maps[2], maps[3], p));
  count_launch();
  const long long items = static_cast<long long>(p.n_seq) * p.Hkv * p.n_mt;
  TRISPEC_CUDA_OK(launch_dependent(verify_attn_pieces_merge_kernel, static_cast<unsigned>(items * AP_MERGE_BLOCKS), AP_MERGE_THREADS, 0,
                                   st, 1, p));
  count_launch();
  return TRISPEC_OK;
}

}  // namespace trispec
