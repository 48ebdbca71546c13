// Fused verify pass: tree mask -> attention -> LM-head statistics -> acceptance scan on one
// stream (one verification round of Algorithm 1 for one verifier).
#include "host_common.h"

extern "C" int trispec_verify(const trispec_tree_args* tree, const trispec_attn_args* attn,
                              const trispec_lmhead_args* lm, const trispec_scan_args* scan, void* stream) {
  if (!tree || !lm || !scan) return TRISPEC_ERR_INVALID_ARG;
  int rc = trispec_build_tree_mask(tree, stream);
  if (rc != TRISPEC_OK) return rc;
  if (attn) {
    rc = trispec_verify_attn(attn, stream);
    if (rc != TRISPEC_OK) return rc;
  }
  rc = trispec_lmhead_stats(lm, stream);
  if (rc != TRISPEC_OK) return rc;
  return trispec_accept_scan(scan, stream);
}
