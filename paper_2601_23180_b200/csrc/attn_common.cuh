// Declarations shared by the two attention kernels (split-KV CTAs merged inside a thread-block
// cluster or through a workspace: attn.cu; persistent CTAs that walk balanced pieces of the work:
// attn_pieces.cu): tile geometry, shared-memory and tensor-memory layout, the launch parameters.
#pragma once
#include <math.h>

#include "host_common.h"
#include "sm100.cuh"

namespace trispec {

constexpr int AT_BM = 128;      // rows per M tile
constexpr int AT_BN = 64;       // keys per tile (= paged block size)
constexpr int AT_D = 128;
constexpr int AT_STAGES = 3;        // K ring; the V ring has 3 slots with one P buffer, 2 with two
constexpr int AT_BOX_BYTES = 64 * 64 * 2;               // 64 rows x 64 elements
constexpr int AT_KV_STAGE_BYTES = 4 * AT_BOX_BYTES;     // one K slot + one V slot = 32 KB
constexpr int AT_TILE_BYTES = 2 * AT_BOX_BYTES;         // a K tile or a V tile: 64 keys x 128 dims bf16 = 16 KB
constexpr int AT_P_BYTES = AT_BM * AT_BN * 2;           // 16 KB
constexpr int AT_THREADS = 192;
constexpr int AT_SMEM_USED = AT_STAGES * AT_KV_STAGE_BYTES + AT_P_BYTES + 256;
// two CTAs per SM: 2 x (dynamic + 1 KB reserved) must fit 228 KB, which leaves 768 bytes of alignment slack
constexpr int AT_SMEM_BYTES = AT_SMEM_USED + 768;
constexpr int AT_TMEM_COLS = 256;                        // Q [0,64) S [64,128) O [128,256)
constexpr int AT_TM_Q = 0, AT_TM_S = 64, AT_TM_O = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;                // log2 units
constexpr int AT_PART_PITCH = AT_D * 2 + 16;             // bytes per row of the in-smem partial (bf16, bank spread)
constexpr int AT_PART_ML_OFF = AT_BM * AT_PART_PITCH;    // (m, l) pairs follow the partial rows
constexpr int AT_PART_ML2_OFF = AT_PART_ML_OFF + AT_BM * 8;   // gathered (m, l) of every split for this CTA's rows
constexpr int AT_PART_ML2_MAX = AT_BM + 2 * 8;                // n_splits x rows per CTA, rows rounded up to even
static_assert(AT_PART_ML2_OFF + AT_PART_ML2_MAX * 8 <= (AT_STAGES + 2) * AT_TILE_BYTES,
              "partial must fit in the K ring plus the shorter V ring");

struct AttnParams {
  int T, Hq, Hkv, G, NPT, n_mt, n_splits;
  int paged, max_blocks_per_seq, num_blocks;
  int Lcap;         // capacity of a sequence's context: Lmax, or 64 x max_blocks_per_seq
  float scale_log2;
  const uint16_t* q;
  const int32_t *block_table, *ctx_len, *seq_index;
  const int32_t* n_nodes;   // tree nodes per sequence (a pruned tree), or null = T
  const uint64_t* mask;
  float* part_o;    // [items][128][128]   (workspace mode only)
  float* part_ml;   // [items][128][2]
  uint16_t* o;      // bf16 [B][T][Hq][128]  (cluster mode writes the result itself)
  float* lse;       // [B][Hq][T] or null
  int32_t* dev_status;
  // persistent kernel only
  int n_seq;        // active sequences (at most 128)
  int n_cta;        // CTAs of the launch: CTA c walks tiles [c W / n_cta, (c + 1) W / n_cta) of the work
};

__device__ __forceinline__ uint4 ld_cluster_u4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared::cluster.v4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
  return v;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

}  // namespace trispec

// the persistent form (attn_pieces.cu)
namespace trispec {
constexpr int AT_PIECES_MAX_SEQ = 128;          // sequences its device-side partition holds
size_t attn_pieces_workspace(int n_cta);
int attn_launch_pieces(AttnParams p, const CUtensorMap* maps /* k, v, k_tree, v_tree */, bool two_p, void* workspace,
                       cudaStream_t st);
}  // namespace trispec
