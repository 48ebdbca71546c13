// Fused verify pass: tree mask -> attention -> LM-head statistics -> acceptance scan on one
// stream (one verification round of Algorithm 1 for one verifier).
#include <mutex>
#include <stdlib.h>

#include "host_common.h"

namespace trispec {
// Side stream and events of trispec_verify_host, one set per device, created on first use.
struct HostPassStreams {
  cudaStream_t copy = nullptr;
  cudaEvent_t fork = nullptr, copied = nullptr, inputs = nullptr;
  bool ready = false;
  std::mutex enqueue;   // the stream and the events are shared by every caller on this device
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
    if (cudaEventCreateWithFlags(&h.inputs, cudaEventDisableTiming) != cudaSuccess) return TRISPEC_ERR_CUDA;
    h.ready = true;
  }
  *out = &h;
  return TRISPEC_OK;
}
}  // namespace trispec

namespace trispec {
// How a pass arranges its attention and its LM head (they do not depend on each other).
enum PassForm { PASS_ATTENTION_FIRST = 0, PASS_LM_FIRST = 1, PASS_SIDE_BY_SIDE = 2 };
static PassForm pass_form(const trispec_attn_args* attn, const trispec_lmhead_args* lm, const trispec_scan_args* scan,
                          int* attn_ctas_out) {
  const int lm_seqs = lm->seq_index ? lm->B_active : lm->B;
  const int attn_ctas = attn ? attn_planned_ctas(attn) : 0;
  if (attn_ctas_out) *attn_ctas_out = attn_ctas;
  if (!attn || lm_seqs != 1 || attn_ctas <= 0) return PASS_ATTENTION_FIRST;
  // TRISPEC_PASS_FORM = attention_first | lm_first | side_by_side overrides the rule below for one active
  // sequence (a tuning and testing aid, read at every call; side by side still needs at most SMs / 2 CTAs)
  if (const char* e = getenv("TRISPEC_PASS_FORM")) {
    if (e[0] == 'a') return PASS_ATTENTION_FIRST;
    if (e[0] == 'l') return PASS_LM_FIRST;
    if (e[0] == 's' && attn_ctas * 2 <= device_sm_count() &&
        !(attn->seq_index && scan && scan->esc_index == attn->seq_index)) return PASS_SIDE_BY_SIDE;
  }
  // not side by side when the scan's escalation list is written over the index list the attention reads:
  // in stream order the scan comes last, side by side it would not
  const bool in_place_list = attn->seq_index && scan && scan->esc_index == attn->seq_index;
  // Side by side the LM head gives up one SM per attention CTA and takes SMs / (SMs - CTAs) times as long;
  // one after the other the pass pays the attention (15-25 us at these sizes) and a launch boundary. With the
  // LM head's time estimated as its bytes of W at 5 TB/s, side by side wins while that extra time stays below
  // about 40 us (measured on one sequence: 32000 x 2048 weights with 16 and 64 CTAs, 151936 x 2048 with 16 and
  // 32 CTAs win; 151936 x 2048 with 64 CTAs loses 180 against 152 us; 128256 x 4096 with 32 CTAs is even).
  // Otherwise the LM head goes first: behind the attention it would stall as a programmatic dependent.
  const int sms = device_sm_count();
  const double lm_us = static_cast<double>(lm->V) * lm->d * 2.0 / 5.0e6;
  if (attn_ctas * 2 <= sms && !in_place_list && lm_us * attn_ctas <= 40.0 * (sms - attn_ctas)) return PASS_SIDE_BY_SIDE;
  return PASS_LM_FIRST;
}
}  // namespace trispec

extern "C" const char* trispec_verify_plan(const trispec_attn_args* attn, const trispec_lmhead_args* lm,
                                           const trispec_scan_args* scan) {
  if (!lm) return "none";
  switch (trispec::pass_form(attn, lm, scan, nullptr)) {
    case trispec::PASS_LM_FIRST: return "lm_first";
    case trispec::PASS_SIDE_BY_SIDE: return "side_by_side";
    default: return "attention_first";
  }
}

extern "C" int trispec_verify(const trispec_tree_args* tree, const trispec_attn_args* attn,
                              const trispec_lmhead_args* lm, const trispec_scan_args* scan, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  if (!tree || !lm || !scan) return TRISPEC_ERR_INVALID_ARG;
  // The attention and the LM head do not depend on each other, so their order is free. A kernel launched as
  // a programmatic dependent gets its launch latency and prologue hidden, but its loads make almost no
  // progress while the kernel before it still runs (measured: the stages of the single-sequence LM head
  // arrive within a microsecond of the attention's end, whenever it started). For one active sequence the
  // LM head is a pure stream of W and loses more behind an attention than the hidden latency is worth (one
  // sequence of 4096 context tokens: 166 us against 156 us the other way round), so there the LM head goes
  // first, or the two run side by side (pass_form above).
  int attn_ctas = 0;
  const trispec::PassForm form = trispec::pass_form(attn, lm, scan, &attn_ctas);
  const bool lm_first = form == trispec::PASS_LM_FIRST;
  int rc;
  // One active sequence and an attention small enough beside the LM head (pass_form): the two run side by
  // side. Mask and attention go to a second stream behind an event recorded on `stream` at the
  // start of the call; the LM head, whose grid is one persistent CTA per SM, leaves them one SM per attention
  // CTA and starts at once, the scan follows it, and `stream` then waits for the second stream: everything
  // the call enqueues is complete before anything enqueued on `stream` after it.
  if (form == trispec::PASS_SIDE_BY_SIDE) {
    using namespace trispec;
    HostPassStreams* hs = nullptr;
    rc = host_pass_streams(&hs);
    if (rc != TRISPEC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    std::unique_lock<std::mutex> enqueue_lock(hs->enqueue);
    TRISPEC_CUDA_OK(cudaEventRecord(hs->fork, st));
    TRISPEC_CUDA_OK(cudaStreamWaitEvent(hs->copy, hs->fork, 0));
    rc = trispec_build_tree_mask(tree, hs->copy);          // ordinary launch: first kernel of the call
    if (rc != TRISPEC_OK) return rc;
    rc = trispec_verify_attn(attn, hs->copy);              // dependent of the mask kernel
    if (rc != TRISPEC_OK) return rc;
    TRISPEC_CUDA_OK(cudaEventRecord(hs->copied, hs->copy));
    entry_scope_next_launch_ordinary();                    // first kernel on `stream`
    lm_reserve_sms_once(attn_ctas);
    rc = trispec_lmhead_stats(lm, stream);
    lm_reserve_sms_once(0);
    if (rc != TRISPEC_OK) return rc;
    rc = trispec_accept_scan(scan, stream);                // dependent of the LM head's last kernel
    if (rc != TRISPEC_OK) return rc;
    TRISPEC_CUDA_OK(cudaStreamWaitEvent(st, hs->copied, 0));
    return TRISPEC_OK;
  }
  rc = trispec_build_tree_mask(tree, stream);
  if (rc != TRISPEC_OK) return rc;
  if (attn && !lm_first) {
    rc = trispec_verify_attn(attn, stream);
    if (rc != TRISPEC_OK) return rc;
  }
  rc = trispec_lmhead_stats(lm, stream);
  if (rc != TRISPEC_OK) return rc;
  if (lm_first) {
    rc = trispec_verify_attn(attn, stream);
    if (rc != TRISPEC_OK) return rc;
  }
  return trispec_accept_scan(scan, stream);
}

// The host-buffer form of the pass. The LM head needs only h (and the tree), the attention
// needs q and the tree keys/values: the latter are copied on a side stream while the LM-head
// GEMM, the longest step, already runs, and the attention follows the GEMM. The caller's
// stream sees one ordered unit of work: everything enqueued here completes before anything
// the caller enqueues on `stream` afterwards.
extern "C" int trispec_verify_host(const trispec_host_io* io, const trispec_tree_args* tree,
                                   const trispec_attn_args* attn, const trispec_lmhead_args* lm,
                                   const trispec_scan_args* scan, void* stream) {
  trispec::EntryScope entry_scope;   // the first kernel launched below is an ordinary launch
  using namespace trispec;
  if (!io || !tree || !lm || !scan) return TRISPEC_ERR_INVALID_ARG;
  // the copies below land in the buffers the structs name: they must describe one and the same pass
  if (tree->parent != lm->parent || tree->parent != scan->parent || lm->tok != scan->tok)
    return TRISPEC_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t BT = static_cast<size_t>(tree->B) * tree->T;
  // A copy list is issued with neighbours merged: requests whose source AND destination follow
  // each other in memory become one transfer (each transfer costs a few microseconds of set-up
  // whatever its size, and a pass moves eleven arrays). Callers get this by carving the arrays
  // out of one host and one device buffer in the order used here.
  struct CopyReq { void* dst; const void* src; size_t bytes; };
  auto copy_list = [](CopyReq* r, int n, cudaMemcpyKind kind, cudaStream_t s) -> cudaError_t {
    int i = 0;
    while (i < n) {
      if (!r[i].dst || !r[i].src || r[i].bytes == 0) { ++i; continue; }
      size_t bytes = r[i].bytes;
      int j = i + 1;
      while (j < n && r[j].dst && r[j].src &&
             static_cast<const char*>(r[j].dst) == static_cast<const char*>(r[i].dst) + bytes &&
             static_cast<const char*>(r[j].src) == static_cast<const char*>(r[i].src) + bytes) {
        bytes += r[j].bytes;
        ++j;
      }
      cudaError_t e = cudaMemcpyAsync(r[i].dst, r[i].src, bytes, kind, s);
      if (e != cudaSuccess) return e;
      i = j;
    }
    return cudaSuccess;
  };
  HostPassStreams* hs = nullptr;
  std::unique_lock<std::mutex> enqueue_lock;
  if (attn) {
    int rc = host_pass_streams(&hs);
    if (rc != TRISPEC_OK) return rc;
    // one caller at a time records and waits on the shared events (host threads driving
    // different streams of one device would otherwise pick up each other's records)
    enqueue_lock = std::unique_lock<std::mutex>(hs->enqueue);
    // the side stream may not overwrite q / k_tree / v_tree before earlier work on `stream`
    // (a previous pass reading them) is done
    TRISPEC_CUDA_OK(cudaEventRecord(hs->fork, st));
  }
  // what the LM head needs goes first through the copy engine
  {
    CopyReq in[3] = {{const_cast<int32_t*>(tree->parent), io->parent, BT * 4},
                     {const_cast<int32_t*>(lm->tok), io->tok, BT * 4},
                     {const_cast<void*>(lm->h), io->h, BT * static_cast<size_t>(lm->d) * 2}};
    TRISPEC_CUDA_OK(copy_list(in, 3, cudaMemcpyHostToDevice, st));
  }
  int attn_ctas = 0;
  const bool side_by_side = pass_form(attn, lm, scan, &attn_ctas) == PASS_SIDE_BY_SIDE;
  if (side_by_side) TRISPEC_CUDA_OK(cudaEventRecord(hs->inputs, st));
  if (attn) {
    TRISPEC_CUDA_OK(cudaStreamWaitEvent(hs->copy, hs->fork, 0));
    CopyReq in[3] = {{const_cast<void*>(attn->q), io->q, BT * static_cast<size_t>(attn->Hq) * attn->D * 2},
                     {const_cast<void*>(attn->k_tree), io->k_tree, BT * static_cast<size_t>(attn->Hkv) * attn->D * 2},
                     {const_cast<void*>(attn->v_tree), io->v_tree, BT * static_cast<size_t>(attn->Hkv) * attn->D * 2}};
    TRISPEC_CUDA_OK(copy_list(in, 3, cudaMemcpyHostToDevice, hs->copy));
    if (!side_by_side) TRISPEC_CUDA_OK(cudaEventRecord(hs->copied, hs->copy));
  }
  int rc;
  if (side_by_side) {
    // one active sequence, short context (as in trispec_verify): mask and attention follow their inputs on
    // the second stream, the LM head and the scan run on `stream`, which then waits for the second stream
    TRISPEC_CUDA_OK(cudaStreamWaitEvent(hs->copy, hs->inputs, 0));   // the tree's parents have arrived
    rc = trispec_build_tree_mask(tree, hs->copy);
    if (rc != TRISPEC_OK) return rc;
    rc = trispec_verify_attn(attn, hs->copy);
    if (rc != TRISPEC_OK) return rc;
    TRISPEC_CUDA_OK(cudaEventRecord(hs->copied, hs->copy));
    entry_scope_next_launch_ordinary();                              // first kernel on `stream`
    lm_reserve_sms_once(attn_ctas);
    rc = trispec_lmhead_stats(lm, stream);
    lm_reserve_sms_once(0);
    if (rc != TRISPEC_OK) return rc;
    rc = trispec_accept_scan(scan, stream);
    if (rc != TRISPEC_OK) return rc;
    TRISPEC_CUDA_OK(cudaStreamWaitEvent(st, hs->copied, 0));
  } else {
    rc = trispec_build_tree_mask(tree, stream);
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
  }
  const size_t B = static_cast<size_t>(scan->B);
  CopyReq out[5] = {{io->accept_len, scan->accept_len, B * 4},
                    {io->bonus_tok, scan->bonus_tok, B * 4},
                    {io->last_node, scan->last_node, B * 4},
                    {io->path, scan->path, B * static_cast<size_t>(scan->T) * 4},
                    {io->escalate, scan->escalate, B}};
  TRISPEC_CUDA_OK(copy_list(out, 5, cudaMemcpyDeviceToHost, st));
  return TRISPEC_OK;
}
