/*
 * trispec.h — C ABI of the B200 (sm_100a) verify pass of TriSpec, ternary speculative
 * decoding with a lightweight proxy verifier.
 *
 * One verification pass scores a draft tree of T = k + 1 nodes per sequence (node 0 is the
 * last committed token, whose output distribution is p_1 of Eq. 2 / Eq. 5; nodes 1..k are the
 * k drafted tokens). The pass is:
 *   1. trispec_build_tree_mask  ancestor mask of the draft tree (Figure 4, Section 4.1)
 *   2. trispec_verify_attn      GQA attention of the tree tokens over the committed KV cache
 *                               and the tree's own keys under that mask (Eq. 2 / Eq. 5)
 *   3. trispec_lmhead_stats     LM head fused with per-position softmax statistics: max,
 *                               log-sum-exp, top_1 / top_2 (Eq. 8), p(drafted token) (Eq. 6)
 *   4. trispec_accept_scan      acceptance length tau_a (Eq. 7), trusted prefix tau_m (Eq. 9)
 *                               and routing: approve or escalate (cases (i)/(ii), Algorithm 1)
 *   trispec_verify              the four in order on one stream.
 * Around the pass, for the decode loop:
 *   5. trispec_prune_tree       the branches that remain for the target after the proxy
 *                               accepted a prefix (routing case (ii), token pruning)
 *   6. trispec_commit_kv        append the accepted path's keys/values to the KV cache
 *   7. trispec_sample_bonus     draw the bonus token from a node's distribution (temperature 1)
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer owned by the caller unless a comment says
 *     "host". The library never frees or retains caller memory past the call.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default
 *     stream). No call synchronises the device.
 *   - Return value: 0 (TRISPEC_OK) or a trispec_status error. Argument errors are detected
 *     on the host before anything is launched. No exceptions, no output on stdout/stderr.
 *   - bf16 tensors are passed as `const void*` (16-bit patterns). D (head dim) must be 128,
 *     T <= 64, Hq / Hkv in {1, 2, 4, 8, 16}.
 *   - Rows of per-node arrays are indexed row = b * T + node.
 *   - `dev_status` (optional, int32 on the device, caller zeroes it): receives a non-zero
 *     trispec_status code when a kernel meets a condition it has to work around (a bounded wait
 *     that gave up, an index or length outside its range, a malformed tree); the kernels never
 *     trap and never read or write outside the caller's arrays because of such a value.
 *   - Ordering. A call may read any of its inputs as soon as its first kernel starts, and that
 *     kernel is an ordinary stream-ordered launch: whatever was enqueued on `stream` before the
 *     call - the caller's own kernels and copies, or an earlier call of this library such as a
 *     KV commit, a pruning step or the scan that wrote an escalation list - has completed by
 *     then. One exception is the caller's to avoid: a kernel that uses programmatic dependent
 *     launch and signals completion before its last write to q, k_tree, v_tree, h, the KV
 *     cache or an index array must not be the last thing on the stream before a call.
 *     Inside one call the library's kernels overlap their prologues and tails (programmatic
 *     dependent launch); seen from the stream a call is one ordered unit of work.
 */
#ifndef TRISPEC_H_
#define TRISPEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  TRISPEC_OK = 0,
  TRISPEC_ERR_INVALID_ARG = 1,     /* null pointer, non-positive size, misaligned pointer */
  TRISPEC_ERR_UNSUPPORTED = 2,     /* D != 128, T > 64, unsupported group size, ... */
  TRISPEC_ERR_WORKSPACE = 3,       /* workspace_bytes smaller than the *_workspace() query */
  TRISPEC_ERR_CUDA = 4,            /* a CUDA runtime / driver call failed */
  TRISPEC_ERR_DEVICE_TIMEOUT = 5,  /* dev_status: a bounded device-side wait gave up; results are invalid */
  TRISPEC_ERR_BAD_BLOCK = 6,       /* dev_status: block_table entry outside [0, num_blocks), read as block 0 */
  TRISPEC_ERR_SMEM_ALIGN = 7,      /* dev_status: a kernel's shared-memory window was not where it must be */
  TRISPEC_ERR_TOO_LARGE = 8,       /* problem needs more than the library's built-in scratch */
  TRISPEC_ERR_NO_ROOM = 9,         /* dev_status: a KV commit would exceed a sequence's capacity; skipped */
  TRISPEC_ERR_BAD_LENGTH = 10,     /* dev_status: ctx_len[b] outside [0, capacity], clamped to it */
  TRISPEC_ERR_BAD_TREE = 11        /* dev_status: parent[] of some sequence is not a tree (see entry 1) */
} trispec_status;

#define TRISPEC_MODE_PROXY 0   /* margin rule of Eq. 8-9 applied (proxy verifier) */
#define TRISPEC_MODE_TARGET 1  /* plain left-to-right acceptance (target verifier, after Eq. 10) */

/* routing criteria (Section "Routing Criteria"): a position is trusted iff */
#define TRISPEC_CRIT_MARGIN 0   /* p_top1 - p_top2 >= lambda (Eq. 8; the paper's default) */
#define TRISPEC_CRIT_TOP1 1     /* p_top1 >= lambda */
#define TRISPEC_CRIT_ENTROPY 2  /* entropy <= lambda (plain Shannon entropy in nats) */

/* acceptance rules: a drafted child c of the current node is accepted iff */
#define TRISPEC_ACCEPT_GREEDY 0          /* tok[c] is the arg-max token (greedy form of Eq. 6) */
#define TRISPEC_ACCEPT_STOCHASTIC 1      /* u < min(1, p(tok[c]) / q(tok[c])) (Eq. 6 at temperature 1) */
#define TRISPEC_ACCEPT_TOKEN_SPECIFIC 2  /* p(tok[c]) >= (1 - alpha) * max p (token-specific deferral
                                            rule, appendix "Baseline Implementation Details: SpecCascade") */

#define TRISPEC_KV_CONTIGUOUS 0 /* k_cache, v_cache: [B][Lmax][Hkv][D] */
#define TRISPEC_KV_PAGED 1      /* pool [num_blocks][block_size][Hkv][D] + block_table */

const char* trispec_status_string(int status);

/* Number of the library's own kernels launched on this process since load (host counter). */
long long trispec_launch_count(void);

/* ---------------------------------------------------------------------------------------
 * 1. Tree mask (Figure 4 "attention mask updates"; draft tree of Section 4.1).
 *    parent [B][T] int32: parent[b][0] = -1, 0 <= parent[b][i] < i.
 *    mask   [B][T] uint64: bit j of mask[b][i] is 1 iff j is an ancestor of i or j == i.
 *    depth  [B][T] int32 : edges from the root (may be NULL).
 *    Malformed parents (>= i or < -1, or parent[b][0] != -1) are not dereferenced: the node and
 *    every node below it get mask 0 and depth -1 (such a node attends to no tree key),
 *    and dev_status (optional) receives TRISPEC_ERR_BAD_TREE, which is
 *    how a caller of the fused pass learns of it after the pass.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  int B, T;
  const int32_t* parent;
  uint64_t* mask;
  int32_t* depth;
  int32_t* dev_status;
} trispec_tree_args;
int trispec_build_tree_mask(const trispec_tree_args* a, void* stream);

/* ---------------------------------------------------------------------------------------
 * 2. Verification attention (the attention of the parallel verification pass, Eq. 2 / 5).
 *    o[b][i][h] = sum_j softmax_j(scale * q[b][i][h] . k_j) v_j over all ctx_len[b] context
 *    keys plus the tree keys j with bit j set in mask[b][i]; KV head of h is h / (Hq/Hkv).
 *    q [B][T][Hq][D], k_tree/v_tree [B][T][Hkv][D], o [B][T][Hq][D]: bf16.
 *    kv_layout CONTIGUOUS: k_cache/v_cache [B][Lmax][Hkv][D] bf16.
 *    kv_layout PAGED: pool [num_blocks][block_size=64][Hkv][D]; token t of sequence b is in
 *      block block_table[b][t / 64] (int32 [B][max_blocks_per_seq]), slot t % 64.
 *    ctx_len [B] int32, 0 <= ctx_len[b] <= Lmax (contiguous) or 64 * max_blocks_per_seq; a
 *      value outside that range is clamped to it and dev_status receives TRISPEC_ERR_BAD_LENGTH.
 *    seq_index (optional, int32 [B_active], device): only these sequences are computed;
 *      NULL = all B (then B_active is ignored).
 *    lse (optional) f32 [B][Hq][T]: log-sum-exp of the scaled scores.
 *    n_nodes (optional, int32 [B], device): sequence b has only its first n_nodes[b] tree
 *      nodes (a pruned tree: n_keep of trispec_prune_tree, the branches that are passed on to
 *      the target in routing case (ii)); rows o[b][i] and lse of nodes i >= n_nodes[b] are
 *      neither computed nor written, and whole 128-row tiles past them cost nothing. The
 *      mask rows of the remaining nodes must not name nodes >= n_nodes[b]; rows of q, k_tree
 *      and v_tree past the count may hold anything (they are never used). NULL = T nodes.
 *    workspace: device scratch of at least trispec_verify_attn_workspace(a) bytes,
 *      256-byte aligned; contents are undefined before and after the call. The query
 *      returns 0 (and workspace may be NULL) whenever the context is cut into at most 8
 *      key/value splits per sequence, which are then merged on chip; only few sequences
 *      with long contexts need more splits and a workspace.
 *    Pointers of bf16 tensors must be 16-byte aligned.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  int B, T, Hq, Hkv, D;
  float scale;
  const void *q, *k_tree, *v_tree;
  int kv_layout;
  const void *k_cache, *v_cache;
  int Lmax, num_blocks, block_size, max_blocks_per_seq;
  const int32_t *block_table, *ctx_len;
  const uint64_t* mask;
  const int32_t* seq_index;
  int B_active;
  void* o;
  float* lse;
  void* workspace;
  size_t workspace_bytes;
  int32_t* dev_status;
  const int32_t* n_nodes;
} trispec_attn_args;
size_t trispec_verify_attn_workspace(const trispec_attn_args* a);
int trispec_verify_attn(const trispec_attn_args* a, void* stream);
/* Which kernels a call with these arguments would take (a diagnostic; host only, nothing is launched):
 * "cluster" = key/value splits merged on chip, "splits" = splits merged through the workspace,
 * "pieces" = persistent CTAs over balanced pieces of the work (long or ragged contexts), "none" =
 * arguments refused. The environment variable TRISPEC_ATTN_PLAN = pieces | splits overrides the choice
 * between the last one and the first two where both apply. */
const char* trispec_verify_attn_plan(const trispec_attn_args* a);

/* ---------------------------------------------------------------------------------------
 * 3. LM-head softmax statistics (distributions p_i in R^V of Eq. 5; top_1, top_2 of Eq. 8).
 *    z[r][v] = logit_scale * <h[r], W[v]>; no [rows x V] logits are written to memory.
 *    Per row r = b*T + node (all arrays [B*T]):
 *      max, lse = log sum_v exp z; (top1_val, top1_idx) largest entry, (top2_val, top2_idx)
 *      largest entry among the other indices (ties -> lowest index);
 *      p_top1 = exp(top1_val - lse), p_top2 likewise; entropy = -sum_v p_v ln p_v (the
 *      feature of the entropy routing criterion, "Routing Criteria" study).
 *    Per CHILD node c >= 1: draft_logit[b*T+c] = z[b*T+parent[c]][tok[c]] and
 *      p_draft = exp(draft_logit - lse[parent row]); entries of node 0 are NaN.
 *    h [B*T][d] bf16, W [V][d] bf16 (row-major, 16-byte aligned, d % 64 == 0).
 * ------------------------------------------------------------------------------------- */
typedef struct {
  float *max, *lse, *top1_val, *top2_val, *p_top1, *p_top2;
  int32_t *top1_idx, *top2_idx;
  float *draft_logit, *p_draft;
  float* entropy;  /* optional (may be NULL): -sum_v p ln p in nats, per row like lse */
} trispec_stats;

typedef struct {
  int B, T, d, V;
  float logit_scale;
  const void *h, *W;
  const int32_t *parent, *tok;
  const int32_t* seq_index;  /* optional subset, as in trispec_attn_args */
  int B_active;
  trispec_stats out;
  void* workspace;           /* >= trispec_lmhead_stats_workspace(a) bytes, 256-byte aligned */
  size_t workspace_bytes;
  int32_t* dev_status;
} trispec_lmhead_args;
size_t trispec_lmhead_stats_workspace(const trispec_lmhead_args* a);
int trispec_lmhead_stats(const trispec_lmhead_args* a, void* stream);

/* ---------------------------------------------------------------------------------------
 * 3b. LM-head statistics for callers that cannot allocate device memory. (The paper has no
 *     counterpart: this is a packaging variant of entry point 3, same inputs, same results.)
 *     A decode loop embedded in a serving engine often runs after the engine has handed all
 *     free device memory to its KV-cache pool; a cudaMalloc there fails or, when it works,
 *     stalls every stream of the process. Such a caller has nowhere to get the per-call
 *     workspace of trispec_lmhead_stats from. This entry point takes none: the per-slice
 *     partial statistics go to a fixed array of TRISPEC_NOALLOC_SCRATCH_BYTES that is part of
 *     the library image (every GPU that loads the library holds that much until the process
 *     exits). `workspace` and `workspace_bytes` of the argument struct are ignored; inputs
 *     and outputs are still the caller's. No device or host memory is allocated or freed.
 *       - Limit: up to 512 active sequences (the partial statistics, planned for this entry
 *         point so that they fit where they can, must not exceed TRISPEC_NOALLOC_SCRATCH_BYTES =
 *         1 MiB); beyond that the call returns TRISPEC_ERR_TOO_LARGE and launches nothing.
 *       - The first call on each device looks up the device address of the array (one
 *         runtime call, with that device current); make that first call outside any stream
 *         capture. Later calls on the device reuse the address.
 *       - All calls on a device share the one array, and it keeps whatever the last call left
 *         in it. Nothing in it needs clearing: a call overwrites every entry it later reads.
 *         Two calls whose kernels overlap on the GPU (different streams) race on it; calls on
 *         one stream are ordered and safe.
 * ------------------------------------------------------------------------------------- */
#define TRISPEC_NOALLOC_SCRATCH_BYTES (1u << 20)
int trispec_lmhead_stats_noalloc(const trispec_lmhead_args* a, void* stream);

/* ---------------------------------------------------------------------------------------
 * 4. Acceptance scan (Eq. 6 greedy form, Eq. 7, Eq. 8, Eq. 9, routing cases (i)/(ii),
 *    Algorithm 1). Per sequence, walking from start_node (root if NULL):
 *      PROXY mode: if p_top1 - p_top2 < lambda at the current node -> escalate (case (ii),
 *      the accepted tokens so far are x_{1:tau_m}); else the child whose token equals
 *      top1_idx is accepted and the walk continues; no such child -> approve (case (i)),
 *      bonus_tok = top1_idx of the current node. TARGET mode: no margin test.
 *    Stochastic acceptance (Eq. 6 at temperature 1), when q_draft and u_accept (f32 [B][T],
 *      indexed by child node) are given: child c of the current node is accepted iff
 *      u_accept[c] < min(1, in.p_draft[c] / q_draft[c]) (q_draft = the drafter's probability of
 *      tok[c], u_accept = the caller's uniform numbers in [0, 1)); the children are tried in
 *      node order and the first accepted one is taken. When none is accepted the round ends in
 *      case (i) with bonus_tok = -2: the bonus token has to be sampled at last_node
 *      (trispec_sample_bonus). The decision is taken in fp32 (IEEE division).
 *    Token-specific deferral rule (accept_rule = TRISPEC_ACCEPT_TOKEN_SPECIFIC; the rule of the
 *      SpecCascade baselines that looks only at the verifier's distribution; the paper runs it
 *      with alpha = 0.2): child c of the current node is accepted iff
 *      in.p_draft[c] >= (1 - alpha) * in.p_top1[current node], 0 <= alpha <= 1, compared in fp32;
 *      the children are tried in node order and the first that passes is taken; when none
 *      passes the round ends in case (i) with bonus_tok = top1_idx of the current node.
 *      alpha = 0 is greedy acceptance, alpha = 1 accepts any drafted token.
 *    active (optional uint8 [B]): sequences with 0 are skipped (outputs: accept_len 0,
 *      escalate 0, bonus -1, last_node -1, path -1).
 *    Outputs: accept_len, bonus_tok, last_node, near_thr int32 [B]; escalate uint8 [B];
 *      path int32 [B][T] (accepted node ids in order, -1 padded);
 *      near_thr = visited positions with |feature - lambda| < 1e-3 (PROXY mode), the feature
 *      being the margin, p_top1 or the entropy as `criterion` selects;
 *      n_escalated int32 [1]; esc_index int32 [B] ascending ids of escalated sequences,
 *      -1 padded. near_thr, n_escalated and esc_index may be NULL (n_escalated and esc_index
 *      only together). compact_scratch (optional) only changes how fast esc_index is built for
 *      very large batches, never its contents.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  int B, T;
  float lambda;
  int mode;
  int criterion;             /* TRISPEC_CRIT_*: which proxy feature decides trust (0 = margin) */
  const int32_t *parent, *tok;
  trispec_stats in;          /* read: top1_idx, and p_top1, p_top2 or entropy as the criterion needs */
  const uint8_t* active;
  const int32_t* start_node;
  const float *q_draft, *u_accept;  /* both NULL: greedy acceptance; both set: Eq. 6 at temperature 1 */
  int accept_rule;                  /* TRISPEC_ACCEPT_*; GREEDY with q_draft/u_accept set means STOCHASTIC */
  float alpha;                      /* slack of the token-specific rule; ignored by the other rules */
  int32_t *accept_len, *bonus_tok, *path, *last_node, *near_thr, *n_escalated, *esc_index;
  uint8_t* escalate;
  int32_t* compact_scratch;         /* optional, int32 [ceil(B / 65536)], contents undefined: lets batches above
                                       65536 sequences build esc_index with one block per 65536 flags */
} trispec_scan_args;
int trispec_accept_scan(const trispec_scan_args* a, void* stream);

/* ---------------------------------------------------------------------------------------
 * 5. Token pruning (routing case (ii): the accepted tokens are pruned from the draft tree and
 *    the remaining branches go to the target; ablation "Token pruning strategies").
 *    For every sequence with root[b] >= 0 the subtree below node root[b] (the last node the
 *    proxy accepted, `last_node` of the scan) is compacted into a tree of its own: root[b]
 *    becomes node 0, the other kept nodes follow in their old order, so parent'[i] < i holds.
 *      parent, tok [B][T] int32, mask [B][T] uint64 (from trispec_build_tree_mask): inputs.
 *      root [B] int32: node to keep the subtree of; < 0 = skip the sequence (n_keep 0).
 *      n_keep [B] int32: size of the subtree.
 *      node_map [B][T] int32: new index -> old index (the gather list for per-node data of
 *        the old tree), -1 beyond n_keep.
 *      parent_out, tok_out [B][T] int32: the pruned tree, -1 beyond n_keep.
 *      mask_out [B][T] uint64, depth_out [B][T] int32 (either may be NULL): ancestor mask and
 *        depth of the pruned tree (what trispec_build_tree_mask would give for parent_out);
 *        entries beyond n_keep are 0 and -1.
 *    Outputs may not alias inputs.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  int B, T;
  const int32_t *parent, *tok;
  const uint64_t* mask;
  const int32_t* root;
  int32_t *n_keep, *node_map, *parent_out, *tok_out;
  uint64_t* mask_out;
  int32_t* depth_out;
} trispec_prune_args;
int trispec_prune_tree(const trispec_prune_args* a, void* stream);

/* ---------------------------------------------------------------------------------------
 * 6. KV commit (X <- X + Y of Algorithm 1 as the KV cache sees it). Appends, for every
 *    active sequence, the keys/values of tree node 0 (the last committed token, not in the
 *    cache yet) and of the accept_len[b] accepted nodes path[b][0..accept_len[b]) to the
 *    sequence's cache at positions ctx_len[b], ctx_len[b] + 1, ..., and writes the new length.
 *      k_tree, v_tree [B][T][Hkv][D] bf16; path [B][T], accept_len [B] (outputs of the scan).
 *      k_cache, v_cache: the cache to append to, layouts as in trispec_verify_attn
 *        (contiguous [B][Lmax][Hkv][D], or paged pool + block_table).
 *      ctx_len [B] int32: current lengths; ctx_len_out [B] int32: lengths after the commit
 *        (may be the same pointer as ctx_len: updated in place).
 *      active (optional uint8 [B]): 0 = leave the sequence alone.
 *    A sequence whose new length would exceed its capacity (Lmax, or 64 x the number of
 *    non-negative entries at the head of its block_table row) is left unchanged and
 *    dev_status (optional) receives 9. D = 128 only.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  int B, T, Hkv, D;
  const void *k_tree, *v_tree;
  int kv_layout;
  void *k_cache, *v_cache;
  int Lmax, num_blocks, block_size, max_blocks_per_seq;
  const int32_t* block_table;
  const int32_t *ctx_len, *path, *accept_len;
  const uint8_t* active;
  int32_t* ctx_len_out;
  int32_t* dev_status;
} trispec_commit_args;
int trispec_commit_kv(const trispec_commit_args* a, void* stream);

/* ---------------------------------------------------------------------------------------
 * 7. Bonus sampling (Algorithm 1: x_bonus ~ p_{tau_a + 1}; needed at temperature 1, where the
 *    stochastic scan ends case (i) with bonus_tok = -2). For every sequence whose bonus_tok[b]
 *    equals -2, a token is drawn from softmax(logit_scale * h[b][last_node[b]] . W^T) by the
 *    Gumbel-max identity: argmax_v (z_v + G_v), G_v independent standard Gumbel variates
 *    (ties -> lowest index). The noise is counter-based and reproducible: word (v mod 4) of
 *    Philox-4x32-10 with counter (v div 4, b, step low, step high) and key (seed low, seed high)
 *    gives u = ((word >> 9) + 0.5) / 2^23 and G = -ln(-ln u). (The upper 23 bits of the word: u is
 *    then exact in single precision and never 0 or 1. It bounds the variate to [-2.812, 16.636]:
 *    an entry more than 19.45 below the largest logit, probability under 4e-9, is never drawn.)
 *    One more pass over W, no logits in global memory.
 *      h [B*T][d], W [V][d] bf16 as in trispec_lmhead_stats; last_node [B] int32.
 *      bonus_tok [B] int32, in/out: entries equal to -2 are replaced by the sampled token;
 *        other entries are left alone. sample_value (optional f32 [B]): the winning z_v + G_v.
 *      seed, step: the caller advances `step` every round.
 *      workspace: >= trispec_sample_bonus_workspace(a) bytes, 256-byte aligned.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  int B, T, d, V;
  float logit_scale;
  const void *h, *W;
  const int32_t* last_node;
  int32_t* bonus_tok;
  float* sample_value;
  unsigned long long seed, step;
  void* workspace;
  size_t workspace_bytes;
  int32_t* dev_status;
} trispec_sample_args;
size_t trispec_sample_bonus_workspace(const trispec_sample_args* a);
int trispec_sample_bonus(const trispec_sample_args* a, void* stream);

/* ---------------------------------------------------------------------------------------
 * Fused pass: the four calls above on `stream` (one verification round of Algorithm 1 for
 * one verifier): tree mask first, acceptance scan last; the attention and the LM-head
 * statistics, which do not read each other's results, in the order the library finds faster
 * for the shape. `attn` may be NULL to skip attention. For one active sequence whose attention
 * needs few CTAs the library runs mask + attention on an internal second stream beside the LM head and
 * the scan, and `stream` waits for that stream before the call returns its place in the queue:
 * what the caller sees is unchanged (everything the call enqueues has completed before anything
 * enqueued on `stream` afterwards starts), but no output buffer of the call may overlap an input
 * of another step of the same call (the one case the library checks and serialises itself:
 * scan->esc_index == attn->seq_index).
 * ------------------------------------------------------------------------------------- */
int trispec_verify(const trispec_tree_args* tree, const trispec_attn_args* attn,
                   const trispec_lmhead_args* lm, const trispec_scan_args* scan, void* stream);
/* How a pass with these arguments arranges its attention and its LM head (a diagnostic; host only,
 * nothing is launched; `attn` and `scan` may be NULL): "attention_first" (batches), "lm_first" or
 * "side_by_side" (one active sequence: the second-stream form described above where the LM head can
 * spare the attention's SMs); "none" without `lm`. The environment variable TRISPEC_PASS_FORM =
 * attention_first | lm_first | side_by_side overrides the choice for one active sequence. */
const char* trispec_verify_plan(const trispec_attn_args* attn, const trispec_lmhead_args* lm,
                                const trispec_scan_args* scan);

/* ---------------------------------------------------------------------------------------
 * The same pass for callers whose per-round data lives in HOST memory (one verification
 * round of Algorithm 1 as a decode loop sees it: the draft tree and its activations arrive
 * from the host, the routing decision goes back to it). The KV cache and the LM-head weights
 * stay resident on the device. Copies the per-round inputs from the host pointers of `io`
 * into the device buffers named by the argument structs (tree->parent, lm->tok, lm->h on
 * `stream`; attn->q, attn->k_tree, attn->v_tree on a stream of the library's own, ordered
 * after everything already on `stream`, so that they overlap the LM-head GEMM), runs the
 * tree mask, the LM-head statistics, the attention and the scan, then copies accept_len,
 * escalate, bonus_tok, last_node and path back to the host pointers. Seen from `stream` the
 * call is one ordered unit of work. The first call on a device creates that stream and two
 * events (host resources, kept until the process exits); no device memory is allocated.
 * Host pointers should be page-locked for the copies to be asynchronous; the results are
 * valid once `stream` has been synchronised. NULL host input pointers skip that copy.
 * Copies whose host AND device addresses follow each other are merged into one transfer, in
 * these orders: (parent, tok, h), (q, k_tree, v_tree), (accept_len, bonus_tok, last_node,
 * path, escalate). A caller that carves each group out of one host and one device buffer in
 * that order pays three transfers per round instead of eleven.
 * The device buffers behind tree->parent, lm->tok, lm->h, attn->q, attn->k_tree and
 * attn->v_tree are WRITTEN by this call although the argument structs declare them const (they
 * are inputs of the pass proper). The structs must describe one pass: tree->parent, lm->parent
 * and scan->parent have to be the same pointer, and so do lm->tok and scan->tok; otherwise the
 * call returns TRISPEC_ERR_INVALID_ARG and does nothing.
 * ------------------------------------------------------------------------------------- */
typedef struct {
  const int32_t *parent, *tok;              /* host [B][T] */
  const void *q, *k_tree, *v_tree, *h;      /* host bf16, same layouts as the device tensors */
  int32_t *accept_len, *bonus_tok, *last_node, *path;  /* host outputs [B], [B], [B], [B][T] */
  uint8_t* escalate;                         /* host output [B] */
} trispec_host_io;
int trispec_verify_host(const trispec_host_io* io, const trispec_tree_args* tree,
                        const trispec_attn_args* attn, const trispec_lmhead_args* lm,
                        const trispec_scan_args* scan, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TRISPEC_H_ */
