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

extern "C" int trispec_verify_host(const trispec_host_io* io, const trispec_tree_args* tree,
                                   const trispec_attn_args* attn, const trispec_lmhead_args* lm,
                                   const trispec_scan_args* scan, void* stream) {
  if (!io || !tree || !lm || !scan) return TRISPEC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t BT = static_cast<size_t>(tree->B) * tree->T;
  auto h2d = [&](const void* dst, const void* src, size_t bytes) -> cudaError_t {
    if (!src || !dst) return cudaSuccess;
    return cudaMemcpyAsync(const_cast<void*>(dst), src, bytes, cudaMemcpyHostToDevice, st);
  };
  TRISPEC_CUDA_OK(h2d(tree->parent, io->parent, BT * 4));
  TRISPEC_CUDA_OK(h2d(lm->tok, io->tok, BT * 4));
  TRISPEC_CUDA_OK(h2d(lm->h, io->h, BT * static_cast<size_t>(lm->d) * 2));
  if (attn) {
    TRISPEC_CUDA_OK(h2d(attn->q, io->q, BT * static_cast<size_t>(attn->Hq) * attn->D * 2));
    TRISPEC_CUDA_OK(h2d(attn->k_tree, io->k_tree, BT * static_cast<size_t>(attn->Hkv) * attn->D * 2));
    TRISPEC_CUDA_OK(h2d(attn->v_tree, io->v_tree, BT * static_cast<size_t>(attn->Hkv) * attn->D * 2));
  }
  int rc = trispec_verify(tree, attn, lm, scan, stream);
  if (rc != TRISPEC_OK) return rc;
  auto d2h = [&](void* dst, const void* src, size_t bytes) -> cudaError_t {
    if (!src || !dst) return cudaSuccess;
    return cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, st);
  };
  const size_t B = static_cast<size_t>(scan->B);
  TRISPEC_CUDA_OK(d2h(io->accept_len, scan->accept_len, B * 4));
  TRISPEC_CUDA_OK(d2h(io->bonus_tok, scan->bonus_tok, B * 4));
  TRISPEC_CUDA_OK(d2h(io->last_node, scan->last_node, B * 4));
  TRISPEC_CUDA_OK(d2h(io->path, scan->path, B * static_cast<size_t>(scan->T) * 4));
  TRISPEC_CUDA_OK(d2h(io->escalate, scan->escalate, B));
  return TRISPEC_OK;
}
