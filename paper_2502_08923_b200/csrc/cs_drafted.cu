// CopySpec merged with vanilla speculative decoding (Sec. 3.3; App. B.3 steps 1-4), one
// sequence.  Host code only: every token-level operation runs in the kernels behind
// cs_find_match, cs_verify_step and cs_kv_truncate; this file orders them.
//
//   step:  search the last gamma tokens (step 1)
//          match    -> the k copied tokens are the draft (step 2)
//          no match -> the draft model first runs over the accepted tokens it has not seen
//                      (copy steps leave its cache alone), then proposes delta tokens one at
//                      a time at temperature 0 (step 3(a))
//          the target verifies [last token, draft] in one block, the longest agreeing prefix
//          plus one extra token is emitted (step 3(b); Sec. 3.2), both caches are rolled back
//          to the accepted prefix (step 3(c)), the tokens are appended (step 4)
//
// The host reads the match position and the accepted block back every step, so this loop
// synchronises once or twice per step; the device-resident loop without a draft model is
// cs_decode_loop.  Every forward is replayed from a graph kept per launch shape (the target's
// block, the draft model's catch-up block, its single-row steps).  Scratch: the loop buffers
// of the two contexts' workspaces (CS_MAX_ROWS ints each), so neither context may have a
// cs_loop_begin session open.
#include <algorithm>
#include <cstring>
#include <vector>

#include "cs_common.cuh"

namespace {

cs_status fail2(cs_ctx* ctx, cs_status s, const char* msg) {
  if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s", msg);
  return s;
}

#define DR_CUDA(call)                                                                           \
  do {                                                                                          \
    cudaError_t e__ = (call);                                                                   \
    if (e__ != cudaSuccess) {                                                                   \
      snprintf(target->err, sizeof(target->err), "%s: %s", #call, cudaGetErrorString(e__));     \
      return CS_ERR_CUDA;                                                                       \
    }                                                                                           \
  } while (0)
#define DR_OK(call)                   \
  do {                                \
    cs_status s__ = (call);           \
    if (s__ != CS_OK) return s__;     \
  } while (0)

}  // namespace

extern "C" cs_status cs_decode_loop_drafted(cs_ctx* target, cs_ctx* drafter, int32_t* hist, int32_t* hist_len,
                                            int stride, void* kv_target, int32_t* kv_len_target, void* kv_drafter,
                                            int32_t* kv_len_drafter, int gamma, int k, int delta,
                                            cs_match_policy policy, int max_new, int eos_id, const int32_t* script,
                                            cs_stats* stats_out, uint64_t* draft_stats_out, void* stream) {
  if (target == nullptr) return CS_ERR_ARG;
  if (hist == nullptr || hist_len == nullptr || kv_target == nullptr || kv_len_target == nullptr || gamma < 1 ||
      k < 0 || delta < 0 || max_new < 0 || stride < 1)
    return fail2(target, CS_ERR_ARG, "bad argument");
  if (delta > 0 && (drafter == nullptr || kv_drafter == nullptr || kv_len_drafter == nullptr || drafter == target))
    return fail2(target, CS_ERR_ARG, "delta > 0 needs a draft model context of its own, its cache and its length");
  const int kt = std::max(k, delta);                   // rows of a target block beyond the first
  if (kt > target->cfg.k_max) return fail2(target, CS_ERR_ARG, "k or delta above the target context's k_max");
  if (delta > 0 && drafter->cfg.vocab != target->cfg.vocab)
    return fail2(target, CS_ERR_ARG, "draft model and target must share the vocabulary");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int kd = delta > 0 ? drafter->cfg.k_max : 0;   // the draft model catches up kd + 1 tokens per block

  cs_stats stats;
  memset(&stats, 0, sizeof(stats));
  uint64_t draft_attempts = 0, draft_accepted = 0;
  int n = 0, kvt = 0, d_len = 0;
  DR_CUDA(cudaMemcpyAsync(&n, hist_len, sizeof(int), cudaMemcpyDeviceToHost, st));
  DR_CUDA(cudaMemcpyAsync(&kvt, kv_len_target, sizeof(int), cudaMemcpyDeviceToHost, st));
  if (delta > 0) DR_CUDA(cudaMemcpyAsync(&d_len, kv_len_drafter, sizeof(int), cudaMemcpyDeviceToHost, st));
  DR_CUDA(cudaStreamSynchronize(st));
  if (n < 1 || kvt != n - 1 || (delta > 0 && (d_len < 0 || d_len > n - 1)))
    return fail2(target, CS_ERR_ARG, "lengths inconsistent: kv_len_target must be hist_len - 1 and kv_len_drafter at most that");
  if ((long)n + max_new > stride || (long)n + max_new + kt > target->cfg.max_seq ||
      (delta > 0 && (long)n + max_new + delta > drafter->cfg.max_seq))
    return fail2(target, CS_ERR_CAPACITY, "history row or a KV cache too small for max_new more tokens");

  int32_t* t_mpos = target->loop_mpos;
  int32_t* t_draft = target->loop_draft;
  int32_t* t_dlen = target->loop_dlen;
  int32_t* t_accept = target->loop_accept;
  int32_t* t_out = target->loop_out;
  int32_t* t_argmax = target->loop_argmax;
  int32_t* t_script = target->loop_emitted;            // this step's slice of the script
  int32_t* t_newlen = target->loop_last;
  std::vector<int32_t> out_h((size_t)kt + 1);
  int emitted = 0;
  bool done = false;

  while (emitted < max_new && !done) {
    // ---- step 1: search; the host needs to know whether there was a match
    DR_OK(cs_find_match(hist, hist_len, 1, stride, gamma, k, policy, t_mpos, t_draft, t_dlen, st));
    int mpos = -1;
    DR_CUDA(cudaMemcpyAsync(&mpos, t_mpos, sizeof(int), cudaMemcpyDeviceToHost, st));
    DR_CUDA(cudaStreamSynchronize(st));
    const bool drafted = mpos < 0 && delta > 0;
    if (drafted) {
      // ---- step 3(a): catch up on tokens hist[d_len .. n), forced through in blocks of kd + 1
      // rows (scripted acceptance against the tokens themselves); the last row's greedy token
      // is the first proposal
      int32_t* d_draft = drafter->loop_draft;
      int32_t* d_dlen = drafter->loop_dlen;
      int32_t* d_script = drafter->loop_emitted;
      int32_t* d_accept = drafter->loop_accept;
      int32_t* d_out = drafter->loop_out;
      int32_t* d_argmax = drafter->loop_argmax;
      // (fixed buffers and a fixed block height of kd + 1 rows, rows past the block's tokens dead,
      //  so that every block replays the same graph)
      int32_t* d_last = drafter->loop_last + 1;
      int r = 0;
      while (d_len < n) {
        r = std::min(n - d_len, kd + 1);
        const int dl = r - 1;
        DR_CUDA(cudaMemcpyAsync(d_last, hist + d_len, sizeof(int), cudaMemcpyDeviceToDevice, st));
        // script row: the dl draft tokens, then values that are never looked at by this loop
        DR_CUDA(cudaMemsetAsync(d_script, 0xFF, (size_t)(kd + 1) * 4, st));
        if (dl > 0) {
          DR_CUDA(cudaMemcpyAsync(d_draft, hist + d_len + 1, (size_t)dl * 4, cudaMemcpyDeviceToDevice, st));
          DR_CUDA(cudaMemcpyAsync(d_script, hist + d_len + 1, (size_t)dl * 4, cudaMemcpyDeviceToDevice, st));
        }
        DR_CUDA(cudaMemcpyAsync(d_dlen, &dl, sizeof(int), cudaMemcpyHostToDevice, st));
        DR_OK(cs_verify_step_cached(drafter, d_last, d_draft, d_dlen, 1, kd, kv_drafter, kv_len_drafter, d_script,
                                    d_accept, d_out, d_argmax, st));
        d_len += r;
      }
      DR_CUDA(cudaMemcpyAsync(t_draft, d_argmax + (r - 1), sizeof(int), cudaMemcpyDeviceToDevice, st));
      // the remaining delta - 1 proposals, one single-row greedy step each; the new token is
      // copied into the target's draft row
      // (through one fixed input slot and one fixed output slot, so that all of them replay the same graph)
      int32_t* d_zero = drafter->loop_last + 2;
      int32_t* d_in = drafter->loop_mpos;
      int32_t* d_tok = drafter->loop_mpos + 1;
      const int zero = 0;
      DR_CUDA(cudaMemcpyAsync(d_zero, &zero, sizeof(int), cudaMemcpyHostToDevice, st));
      for (int i = 1; i < delta; ++i) {
        DR_CUDA(cudaMemcpyAsync(d_in, t_draft + (i - 1), sizeof(int), cudaMemcpyDeviceToDevice, st));
        DR_OK(cs_verify_step_cached(drafter, d_in, nullptr, d_zero, 1, 0, kv_drafter, kv_len_drafter, nullptr,
                                    d_accept, d_tok, d_argmax, st));
        DR_CUDA(cudaMemcpyAsync(t_draft + i, d_tok, sizeof(int), cudaMemcpyDeviceToDevice, st));
        d_len += 1;
      }
      DR_CUDA(cudaMemcpyAsync(t_dlen, &delta, sizeof(int), cudaMemcpyHostToDevice, st));
    }
    // ---- steps 2 / 3(b): one target block over [last token, draft]
    const int32_t* script_row = nullptr;
    if (script != nullptr) {
      const int have = std::min(kt + 1, max_new - emitted);   // rows past the script's end cannot be accepted
      DR_CUDA(cudaMemsetAsync(t_script, 0xFF, (size_t)(kt + 1) * 4, st));
      DR_CUDA(cudaMemcpyAsync(t_script, script + emitted, (size_t)have * 4, cudaMemcpyDeviceToDevice, st));
      script_row = t_script;
    }
    int32_t* t_last = target->loop_last + 1;
    DR_CUDA(cudaMemcpyAsync(t_last, hist + (n - 1), sizeof(int), cudaMemcpyDeviceToDevice, st));
    DR_OK(cs_verify_step_cached(target, t_last, t_draft, t_dlen, 1, kt, kv_target, kv_len_target, script_row,
                                t_accept, t_out, t_argmax, st));
    int tau = -1;
    DR_CUDA(cudaMemcpyAsync(&tau, t_accept, sizeof(int), cudaMemcpyDeviceToHost, st));
    DR_CUDA(cudaMemcpyAsync(out_h.data(), t_out, (size_t)(kt + 1) * 4, cudaMemcpyDeviceToHost, st));
    DR_CUDA(cudaStreamSynchronize(st));
    if (tau < 0 || tau > kt) break;                    // the device refused the step; the status word says why
    int c = std::min(tau + 1, max_new - emitted);
    if (script == nullptr && eos_id >= 0) {
      for (int i = 0; i < c; ++i)
        if (out_h[(size_t)i] == eos_id) { c = i + 1; done = true; break; }
    }
    // ---- step 4 and the roll-backs: append, then cut both caches to the accepted prefix
    DR_CUDA(cudaMemcpyAsync(hist + n, t_out, (size_t)c * 4, cudaMemcpyDeviceToDevice, st));
    const int n_new = n + c;
    DR_CUDA(cudaMemcpyAsync(hist_len, &n_new, sizeof(int), cudaMemcpyHostToDevice, st));
    if (c - 1 < tau) {                                 // clipped by max_new or EOS: the step kept tau rows
      const int nl = n_new - 1;
      DR_CUDA(cudaMemcpyAsync(t_newlen, &nl, sizeof(int), cudaMemcpyHostToDevice, st));
      DR_OK(cs_kv_truncate(target, kv_len_target, t_newlen, 1, st));
    }
    if (drafted && d_len > n + c - 1) {                // positions n .. n+c-2 hold accepted proposals
      d_len = n + c - 1;
      DR_CUDA(cudaMemcpyAsync(drafter->loop_last, &d_len, sizeof(int), cudaMemcpyHostToDevice, st));
      DR_OK(cs_kv_truncate(drafter, kv_len_drafter, drafter->loop_last, 1, st));
    }
    n = n_new;
    emitted += c;
    stats.steps += 1;
    stats.emitted += (uint64_t)c;
    if (mpos >= 0) {
      stats.attempts += 1;
      stats.accepted += (uint64_t)(c - 1);
      stats.tau_hist[std::min(c - 1, CS_TAU_HIST - 1)] += 1;
    } else {
      stats.no_match += 1;
      if (drafted) { draft_attempts += 1; draft_accepted += (uint64_t)(c - 1); }
    }
  }
  if (stats_out != nullptr) *stats_out = stats;
  if (draft_stats_out != nullptr) { draft_stats_out[0] = draft_attempts; draft_stats_out[1] = draft_accepted; }
  cs_status s = cs_sync_status(target, st);
  if (delta > 0) {
    const cs_status s2 = cs_sync_status(drafter, st);
    if (s == CS_OK && s2 != CS_OK) {
      snprintf(target->err, sizeof(target->err), "draft model: %s", cs_last_error(drafter));
      s = s2;
    }
  }
  return s;
}
