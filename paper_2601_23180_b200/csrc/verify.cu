// Fused verify pass: tree mask -> attention -> LM-head statistics -> acceptance scan on one
// stream (one verification round of Algorithm 1 for one verifier).
#include <mutex>

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

namespace trispec {
// Side stream and events of trispec_verify_host, one set per device, created on first use.
struct HostPassStreams {
  cudaStream_t copy = nullptr;
  cudaEvent_t fork = nullptr, copied = nullptr;
  bool ready = false;
};
static int host_pass_streams(HostPassStreams** out) {
  static HostPassStreams per_dev[64];
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TRISPEC_ERR_CUDA;
  if (dev < 0 || dev >= 64) return TRISPEC_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(mu);
  HostPassStreams& h = per_dev[dev];
  if (!h.ready) {
    if (cudaStreamCreateWithFlags(&h.copy, cudaStreamNonBlocking) != cudaSuccess) return TRISPEC_ERR_CUDA;
    if (cudaEventCreateWithFlags(&h.fork, cudaEventDisableTiming) != cudaSuccess) return TRISPEC_ERR_CUDA;
    if (cudaEventCreateWithFlags(&h.copied, cudaEventDisableTiming) != cudaSuccess) return TRISPEC_ERR_CUDA;
    h.ready = true;
  }
  *out = &h;
  return TRISPEC_OK;
}
}  // namespace trispec

// The host-buffer form of the pass. The LM head needs only h (and the tree), the attention
// needs q and the tree keys/values: the latter are copied on a side stream while the LM-head
// GEMM, the longest step, already runs, and the attention follows the GEMM. The caller's
// stream sees one ordered unit of work: everything enqueued here completes before anything
// the caller enqueues on `stream` afterwards.
extern "C" int trispec_verify_host(const trispec_host_io* io, const trispec_tree_args* tree,
                                   const trispec_attn_args* attn, const trispec_lmhead_args* lm,
                                   const trispec_scan_args* scan, void* stream) {
  using namespace trispec;
  if (!io || !tree || !lm || !scan) return TRISPEC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t BT = static_cast<size_t>(tree->B) * tree->T;
  auto h2d = [&](const void* dst, const void* src, size_t bytes, cudaStream_t s) -> cudaError_t {
    if (!src || !dst) return cudaSuccess;
    return cudaMemcpyAsync(const_cast<void*>(dst), src, bytes, cudaMemcpyHostToDevice, s);
  };
  HostPassStreams* hs = nullptr;
  if (attn) {
    int rc = host_pass_streams(&hs);
    if (rc != TRISPEC_OK) return rc;
    // the side stream may not overwrite q / k_tree / v_tree before earlier work on `stream`
    // (a previous pass reading them) is done
    TRISPEC_CUDA_OK(cudaEventRecord(hs->fork, st));
  }
  // what the LM head needs goes first through the copy engine
  TRISPEC_CUDA_OK(h2d(tree->parent, io->parent, BT * 4, st));
  TRISPEC_CUDA_OK(h2d(lm->tok, io->tok, BT * 4, st));
  TRISPEC_CUDA_OK(h2d(lm->h, io->h, BT * static_cast<size_t>(lm->d) * 2, st));
  if (attn) {
    TRISPEC_CUDA_OK(cudaStreamWaitEvent(hs->copy, hs->fork, 0));
    TRISPEC_CUDA_OK(h2d(attn->q, io->q, BT * static_cast<size_t>(attn->Hq) * attn->D * 2, hs->copy));
    TRISPEC_CUDA_OK(h2d(attn->k_tree, io->k_tree, BT * static_cast<size_t>(attn->Hkv) * attn->D * 2, hs->copy));
    TRISPEC_CUDA_OK(h2d(attn->v_tree, io->v_tree, BT * static_cast<size_t>(attn->Hkv) * attn->D * 2, hs->copy));
    TRISPEC_CUDA_OK(cudaEventRecord(hs->copied, hs->copy));
  }
  int rc = trispec_build_tree_mask(tree, stream);
  if (rc != TRISPEC_OK) return rc;
  rc = trispec_lmhead_stats(lm, stream);
  if (rc != TRISPEC_OK) return rc;
  if (attn) {
    TRISPEC_CUDA_OK(cudaStreamWaitEvent(st, hs->copied, 0));
    rc = trispec_verify_attn(attn, stream);
    if (rc != TRISPEC_OK) return rc;
  }
  rc = trispec_accept_scan(scan, stream);
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
