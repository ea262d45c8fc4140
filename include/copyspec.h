/*
 * copyspec.h - C ABI of the B200 (sm_100a) copy-and-verify decode step of CopySpec
 * (arXiv 2502.08923, "Accelerating LLMs with Speculative Copy-and-Paste").
 *
 * One decode step is: search the token history for an earlier occurrence of the last
 * gamma tokens and copy the k tokens that followed it as a draft (Sec. 3.1, 3.2); run
 * ONE forward of the target model over [last token, draft] against the KV cache
 * (Sec. 3.2); take the greedy token per row and accept the longest agreeing prefix plus
 * one extra token (Sec. 3.2, App. B.2); drop the KV entries of the rejected tokens
 * (App. B.2, App. B.3 step 2(b)).
 *
 * General conventions
 *   - All pointers are DEVICE pointers unless a parameter says "host".
 *   - Ownership: the caller allocates and frees every buffer (history, lengths, drafts,
 *     KV cache, weights, workspace, outputs).  The library allocates no device memory.
 *     A context keeps the weight and workspace pointers given to cs_create; they must
 *     outlive it.  Other pointers are used only during the call (and by the work the
 *     call enqueued on `stream`).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *     marked "async" only enqueue work.  Work of one context must stay on one stream at
 *     a time (its workspace is shared by consecutive calls).
 *   - Errors: every call returns a cs_status.  Argument errors are found on the host
 *     before anything is launched.  Conditions only the device can see (capacity, a
 *     bounded wait that ran out) are recorded in a device status word that
 *     cs_sync_status returns; the offending sequence is left unmodified.  Nothing traps.
 *   - Integer outputs are bit-reproducible from run to run.
 *
 * Layouts
 *   history    int32 [B][stride]; sequence b holds hist_len[b] accepted tokens: prompt,
 *              earlier turns and everything generated so far (Sec. 3.1).
 *   KV cache   bf16 [n_layers][2 (K then V)][max_batch][n_kv_heads][max_seq][head_dim],
 *              contiguous; K is stored rotated (RoPE applied).  Only positions
 *              [0, kv_len[b]) of sequence b are meaningful (App. B.2).
 *   weights    bf16 row-major [out][in]:  embed [V][d], lm_head [V][d], final_norm [d];
 *              per layer attn_norm [d], wqkv [(H + 2 Hkv) Dh][d] (q rows, k rows, v
 *              rows), wo [d][H Dh], ffn_norm [d], w_down [d][F], and w_gate_up
 *              [ceil(F/64) * 128][d]: blocks of 128 rows, block t holding gate rows
 *              64t..64t+63 followed by up rows 64t..64t+63 (rows past F are zero), so that
 *              one GEMM tile sees both halves of SwiGLU.  All base pointers 16-byte
 *              aligned; d, H*Dh and F multiples of 8.
 *   blocks     a verification block of sequence b has rows r = 0..draft_len[b]:
 *              row 0 is the last accepted token (whose K/V are not cached yet), row r>0
 *              is draft token r-1; row r sits at absolute position kv_len[b] + r.
 *
 * State kept between steps of the loop: hist_len[b] = n counts every accepted token
 * including the last one; kv_len[b] = n - 1.
 *
 * Precision: weights and the KV cache are bf16.  Every activation that enters a tensor-core
 * product (normed activations, rotated queries, softmax weights, attention output, SwiGLU
 * output) is carried as TWO bf16 terms, value = hi + lo, and multiplied twice against the same
 * weight / K / V tile, so activation operands are fp32-equivalent; accumulation, the residual
 * stream, norms, RoPE and softmax are fp32.  Only K/V rows are rounded (to nearest-even bf16)
 * when they are stored in the cache.
 *
 * Environment, read once by cs_create (measurement and test switches; not needed in use):
 *   CS_NO_GRAPH=1          steps are enqueued kernel by kernel instead of replayed from a
 *                          captured CUDA graph (cs_loop_*, cs_step_host, cs_decode_loop_drafted);
 *   CS_ATTN_KERNEL=tc|tcw|mma  forces one attention kernel: tcgen05 with the query rows as the
 *                          M dimension (tc), tcgen05 with the keys and head dims as M (tcw), or
 *                          mma.sync (mma).  Default: by head size, and between the two tcgen05
 *                          kernels by how many key tiles a CTA would walk (tcw from three on,
 *                          unless the block fills the 128 query rows of a tc CTA anyway);
 *   CS_WAIT_LIMIT_US=n     time limit of the kernels' bounded waits in microseconds (default
 *                          2,000,000), see cs_debug_drop_tile.
 */
#ifndef COPYSPEC_H
#define COPYSPEC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cs_ctx cs_ctx; /* opaque; host memory owned by the library */

typedef enum {
  CS_OK = 0,
  CS_ERR_ARG = -1,         /* NULL pointer, negative size, gamma < 1, k > k_max, ...      */
  CS_ERR_SHAPE = -2,       /* model shape the kernels do not support                      */
  CS_ERR_CAPACITY = -3,    /* KV cache, history row or workspace too small                */
  CS_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed (see cs_last_error)       */
  CS_ERR_TIMEOUT = -5,     /* a bounded device-side wait ran out                          */
  CS_ERR_UNSUPPORTED = -6, /* valid request outside what is built                         */
  CS_ERR_LIMIT = -7        /* size beyond the built-in maximum of cs_lm_head_static       */
} cs_status;

/* Which occurrence is used when the last gamma tokens recur more than once.  The paper
 * takes the first one (Sec. 3.2 footnote; App. B.3 step 1(c)); the latest one is the
 * default here. */
typedef enum { CS_MATCH_LATEST = 0, CS_MATCH_FIRST = 1 } cs_match_policy;

typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t max_seq;   /* KV positions per sequence                                        */
  int32_t max_batch; /* sequences per call                                               */
  int32_t k_max;     /* largest draft length; max_batch * (k_max + 1) <= 256             */
  float rope_theta, rms_eps;
} cs_model_config;

typedef struct {
  const void* embed;
  const void* lm_head;
  const void* final_norm;
  /* host arrays of n_layers device pointers each */
  const void* const* attn_norm;
  const void* const* wqkv;
  const void* const* wo;
  const void* const* ffn_norm;
  const void* const* w_gate_up;
  const void* const* w_down;
} cs_weights;

#define CS_TAU_HIST 65
typedef struct {
  uint64_t steps;     /* verification forwards, summed over sequences                    */
  uint64_t attempts;  /* steps that had a match, i.e. a copy attempt                     */
  uint64_t accepted;  /* draft tokens accepted (sum of tau)                              */
  uint64_t emitted;   /* tokens appended to the histories                                */
  uint64_t no_match;  /* steps without a match (plain one-token decode)                  */
  uint64_t tau_hist[CS_TAU_HIST]; /* attempts by accepted length; the last bin also takes
                                     every length beyond CS_TAU_HIST - 1                  */
} cs_stats;

/* Bytes of device workspace cs_create needs for this configuration (0 on a bad config).
 * Host-only arithmetic; needs no GPU. */
size_t cs_workspace_bytes(const cs_model_config* cfg);

/* Builds a context.  `cfg` and `weights` are host structs (copied); `workspace` is a
 * 1024-byte aligned device buffer of at least cs_workspace_bytes(cfg) bytes.  Clears the
 * workspace.  Synchronous.  Errors: CS_ERR_ARG, CS_ERR_SHAPE (head_dim not 32, 64 or
 * 128; n_heads not a multiple of n_kv_heads; max_batch*(k_max+1) > 256; dims not
 * multiples of 8), CS_ERR_CAPACITY, CS_ERR_CUDA. */
cs_status cs_create(cs_ctx** out, const cs_model_config* cfg, const cs_weights* weights,
                    void* workspace, size_t workspace_bytes);
void cs_destroy(cs_ctx* ctx);

/* Text of the last host-side error of this context.  With ctx == NULL: the text of the last
 * failed cs_create of this thread (cs_create has no context to leave it in), or "". */
const char* cs_last_error(const cs_ctx* ctx);

/* Waits for `stream`, then returns and clears the device status word of the context:
 * CS_OK, CS_ERR_CAPACITY, CS_ERR_ARG (cs_kv_truncate asked to grow) or CS_ERR_TIMEOUT. */
cs_status cs_sync_status(cs_ctx* ctx, void* stream);

/* Suffix-match search and draft gather (Sec. 3.1; Sec. 3.2; App. B.3 step 1).  Async.
 * For each sequence b with n = hist_len[b]: among all p0 in [0, n - 2 gamma] with
 * hist[b][p0 + j] == hist[b][n - gamma + j] for every j < gamma (exact token equality;
 * the match may not overlap the key, App. B.3 step 1(c)), match_pos[b] is the largest
 * (LATEST) or smallest (FIRST), or -1 if there is none or n < 2 gamma.  The draft is
 * the draft_len[b] = min(k, n - (p0 + gamma)) tokens that follow the match (0 without a
 * match); draft entries past draft_len[b] are set to -1.
 *   hist [B][stride] int32, hist_len [B] int32, match_pos [B], draft [B][k],
 *   draft_len [B].  1 <= gamma <= 8, 0 <= k, B >= 0 (B == 0 is a no-op).
 *   Needs no context and no scratch memory.  Errors: CS_ERR_ARG, CS_ERR_CUDA. */
cs_status cs_find_match(const int32_t* hist, const int32_t* hist_len, int B, int stride,
                        int gamma, int k, cs_match_policy policy, int32_t* match_pos,
                        int32_t* draft, int32_t* draft_len, void* stream);

/* Index of all gamma-grams of the accepted sequences (Sec. 3.1: a hash map from every
 * gamma-token subsequence to where it occurs, O(gamma) work per appended token and per
 * lookup).  An alternative to the scan of cs_find_match whose cost does not grow with the
 * history; results are identical (tokens are compared, not hashes).
 *   index: caller-allocated DEVICE buffer of cs_gram_index_bytes(B, capacity_tokens) bytes,
 *          one table per sequence sized for histories of up to capacity_tokens tokens;
 *   cs_gram_index_reset   empties it (async);
 *   cs_gram_index_update  inserts the gamma-grams that have become admissible since the last
 *          update: starts p <= hist_len[b] - 2*gamma (a match must end before the key starts,
 *          App. B.3 step 1(c)).  Histories only grow; one index serves one gamma.  Async;
 *   cs_find_match_indexed same outputs as cs_find_match for the history lengths of the last
 *          update (call update first whenever tokens were appended).  Async;
 *   cs_gram_index_status  synchronises the stream; CS_ERR_CAPACITY if a table overflowed.
 * Errors on the host: CS_ERR_ARG, CS_ERR_CUDA. */
size_t cs_gram_index_bytes(int B, int capacity_tokens);
cs_status cs_gram_index_reset(void* index, int B, int capacity_tokens, void* stream);
cs_status cs_gram_index_update(void* index, int B, int capacity_tokens, const int32_t* hist,
                               const int32_t* hist_len, int stride, int gamma, void* stream);
cs_status cs_find_match_indexed(const void* index, int B, int capacity_tokens, const int32_t* hist,
                                const int32_t* hist_len, int stride, int gamma, int k,
                                cs_match_policy policy, int32_t* match_pos, int32_t* draft,
                                int32_t* draft_len, void* stream);
cs_status cs_gram_index_status(const void* index, int B, int capacity_tokens, void* stream);

/* Makes the generation loop of this context (cs_decode_loop, cs_loop_*) search through a
 * gamma-gram index instead of scanning the history (Sec. 3.1; App. B.3 step 1 and step 2(d)):
 * cs_loop_begin empties the index and builds it from the histories, every step looks the last
 * gamma tokens up and, after the append, inserts the grams that have become admissible.
 * Results are those of the scan, bit for bit; the cost no longer grows with the history, which
 * pays beyond roughly 100k tokens per sequence.  `index` is a caller-allocated DEVICE buffer of
 * cs_gram_index_bytes(B, capacity_tokens) bytes for the B the loop will run with;
 * capacity_tokens must be at least the loop's `stride` (CS_ERR_CAPACITY from cs_loop_begin
 * otherwise).  A table that overflows all the same is reported as CS_ERR_CAPACITY by
 * cs_loop_poll / cs_decode_loop.  index == NULL goes back to the scan.  Not while a loop is
 * in progress. */
cs_status cs_set_match_index(cs_ctx* ctx, void* index, int capacity_tokens);

/* One verification forward plus acceptance (Sec. 3.2; App. B.2; App. B.3 step 2). Async.
 * Evaluates the block [last_tok[b], draft[b][0 .. draft_len[b])] of every sequence at
 * positions kv_len[b].. in one forward, appends the block's K/V rows to the cache,
 * takes argmax_ids[b][r] = the lowest id with the largest logit of row r (never
 * writing logits to memory unless logits_dbg is given), and accepts
 *   tau = the largest j <= draft_len[b] with draft[b][i] == target[i] for all i < j,
 * where target[r] = argmax_ids[b][r], or target_script[b][r] when target_script is not
 * NULL (scripted-target mode: the forward and argmax are still computed in full, but
 * acceptance follows the given stream).  Outputs: accept_len[b] = tau, out_tokens[b][0..
 * tau] = target[0..tau] (tau accepted tokens and one extra token, Sec. 3.2; the rest of
 * the row is -1), and kv_len[b] += tau + 1, which is the truncation of App. B.2: the
 * cached rows of rejected tokens lie beyond kv_len and are dead.
 *   last_tok [B], draft [B][k], draft_len [B] (0..k), kv_len [B] in/out,
 *   target_script [B][k+1] or NULL, accept_len [B], out_tokens [B][k+1],
 *   argmax_ids [B][k+1] (rows past draft_len[b] are -1),
 *   logits_dbg fp32 [B][k+1][vocab] or NULL.
 * A sequence with kv_len[b] + draft_len[b] + 1 > max_seq is skipped (accept_len -1,
 * nothing modified) and CS_ERR_CAPACITY is recorded in the status word.
 * Errors on the host: CS_ERR_ARG (NULL, B > max_batch, k > k_max). */
cs_status cs_verify_step(cs_ctx* ctx, const int32_t* last_tok, const int32_t* draft,
                         const int32_t* draft_len, int B, int k, void* kv_cache,
                         int32_t* kv_len, const int32_t* target_script, int32_t* accept_len,
                         int32_t* out_tokens, int32_t* argmax_ids, float* logits_dbg,
                         void* stream);

/* One whole step driven from HOST memory (App. B.3 steps 1, 2 and 4; Sec. 3.2), for callers
 * that keep the token histories on the host.  Synchronous: returns when the step is done.
 * Copies the accepted tokens (hist_len_host[b] ints per sequence), the lengths and this step's
 * script rows to the device, runs cs_find_match and cs_verify_step on them, copies the accepted
 * lengths and the emitted tokens back, and appends the tau + 1 emitted tokens of every sequence
 * to hist_host (hist_len_host advances; kv_len advances on the device).
 *   hist_host int32 [B][stride] host (pinned memory makes the copies asynchronous), in/out;
 *   hist_len_host int32 [B] host, in/out; hist_len_host[b] + k + 1 <= stride (CS_ERR_CAPACITY).
 *   hist_dev int32 [B][stride], hist_len_dev int32 [B]: device buffers of the caller that the
 *            call overwrites.  kv_cache / kv_len as in cs_verify_step (kv_len[b] =
 *            hist_len[b] - 1 on entry).
 *   script_host int32 [B][k+1] host or NULL: the target tokens of this step's rows
 *            (scripted-target mode), NULL = real mode.
 *   accept_len_host int32 [B], out_tokens_host int32 [B][k+1]: host outputs (tau, then the
 *            tau + 1 emitted tokens; -1 beyond).  A sequence the device skipped for lack of
 *            cache room has accept_len -1, is left as it was, and cs_sync_status reports it.
 * Only what the device does not have yet crosses the bus: the call remembers how many tokens
 * of each row it has uploaded to hist_dev, and while the same hist_host / hist_dev pair comes
 * back with every row exactly as long as the previous call left it, it uploads just the tokens
 * that call appended.  Anything else (other buffers, B, stride, a length the call did not
 * produce) uploads the rows in full.  A caller that rewrites tokens below hist_len_host[b] in
 * place without changing the length must call cs_step_host_reset first.
 * The kernels of the step are replayed as a CUDA graph that the context keeps while B, k, gamma,
 * the policy, the mode and the device buffers stay the same (first call and every change: one
 * capture).  The context's loop buffers serve as scratch: not to be mixed with an open
 * cs_loop_begin session.  Errors: CS_ERR_ARG / CS_ERR_CAPACITY on the host before any copy, CS_ERR_CUDA. */
cs_status cs_step_host(cs_ctx* ctx, int32_t* hist_host, int32_t* hist_len_host, int B, int stride,
                       int32_t* hist_dev, int32_t* hist_len_dev, void* kv_cache, int32_t* kv_len,
                       int gamma, int k, cs_match_policy policy, const int32_t* script_host,
                       int32_t* accept_len_host, int32_t* out_tokens_host, void* stream);

/* Forget what cs_step_host has uploaded: its next call uploads the histories in full. */
void cs_step_host_reset(cs_ctx* ctx);

/* KV truncation to an accepted length (App. B.2; App. B.3 step 2(b)).  Async.
 * kv_len[b] = new_len[b] where 0 <= new_len[b] <= kv_len[b]; otherwise kv_len[b] is
 * left as is and CS_ERR_ARG is recorded in the status word.  The cache is contiguous
 * and indexed by length, so no K/V bytes move. */
cs_status cs_kv_truncate(cs_ctx* ctx, int32_t* kv_len, const int32_t* new_len, int B,
                         void* stream);

/* The generation loop (App. B.3 steps 1, 2 and 4; Sec. 3.2).  Synchronous.
 * Repeats {search, gather, verify, accept, truncate, append} for all B sequences until
 * each has emitted max_new tokens (the last block is clipped) or, in real mode, has
 * emitted eos_id (tokens after it are dropped; eos_id < 0 = none).  On entry the cache
 * must hold positions [0, hist_len[b] - 1) and kv_len[b] = hist_len[b] - 1.  Accepted
 * tokens are appended to hist and hist_len/kv_len advance.  `script` [B][max_new]
 * switches to scripted-target mode: row r of a step is checked against
 * script[b][emitted_b + r]; the emitted stream then equals the script.  k = 0 gives
 * plain one-token decoding from the same kernels.
 *   stats_out: host pointer or NULL.  stride >= hist_len[b] + max_new and
 *   max_seq >= hist_len[b] + max_new + k are required, and kv_len[b] == hist_len[b] - 1
 *   (checked on the device: CS_ERR_CAPACITY / CS_ERR_ARG).  A sequence that fails these
 *   checks is left unmodified and counts as finished; the others run to their end, and the
 *   call then returns that error.
 * Returns the first error among the host checks, CUDA and the device status word; a CUDA
 * error or a bounded wait that ran out ends the loop at once. */
cs_status cs_decode_loop(cs_ctx* ctx, int32_t* hist, int32_t* hist_len, int B, int stride,
                         void* kv_cache, int32_t* kv_len, int gamma, int k,
                         cs_match_policy policy, int max_new, int eos_id,
                         const int32_t* script, cs_stats* stats_out, void* stream);

/* The same loop in pieces, for callers that want to run a fixed number of steps or overlap
 * host work (App. B.3 steps 1, 2, 4; one step = search, gather, verify, accept, truncate,
 * append for all B sequences).  cs_loop_begin takes cs_decode_loop's arguments, checks
 * them, resets the per-sequence counters and statistics and prepares a CUDA graph of one
 * step; the pointers must stay valid until cs_loop_end.  cs_loop_steps enqueues n_steps
 * steps (async; steps of finished sequences do nothing).  cs_loop_poll waits for `stream`,
 * copies the statistics (stats_out host, may be NULL) and the number of finished sequences
 * (n_done_out host, may be NULL) and returns the device status like cs_sync_status.
 * cs_loop_end releases the graph (also done by cs_destroy and by the next cs_loop_begin). */
cs_status cs_loop_begin(cs_ctx* ctx, int32_t* hist, int32_t* hist_len, int B, int stride,
                        void* kv_cache, int32_t* kv_len, int gamma, int k,
                        cs_match_policy policy, int max_new, int eos_id, const int32_t* script,
                        void* stream);
cs_status cs_loop_steps(cs_ctx* ctx, int n_steps, void* stream);
cs_status cs_loop_poll(cs_ctx* ctx, cs_stats* stats_out, int* n_done_out, void* stream);
void cs_loop_end(cs_ctx* ctx);
/* What the most recent step of the loop in progress produced, copied to HOST arrays (any of
 * them may be NULL): the match position and draft length of the search (App. B.3 step 1), the
 * accepted length, the tau + 1 emitted tokens and the greedy token of every block row
 * (App. B.3 step 2; rows past the draft are -1).  match_pos, draft_len, accept_len: [B];
 * out_tokens, argmax_ids: [B][k+1].  Waits for `stream`.  Entries of a sequence that had
 * already finished before that step keep the values of its own last step. */
cs_status cs_loop_last_step(cs_ctx* ctx, int32_t* match_pos_host, int32_t* draft_len_host,
                            int32_t* accept_len_host, int32_t* out_tokens_host,
                            int32_t* argmax_ids_host, void* stream);
/* Kernel launches in one step of the loop in progress (nodes of its graph; 0 if none). */
int cs_loop_launches_per_step(const cs_ctx* ctx);

/* CopySpec merged with vanilla speculative decoding (Sec. 3.3; App. B.3 steps 1-4), for ONE
 * sequence.  Synchronous.  Every step searches the last gamma tokens; with a match the k
 * copied tokens are the draft, without one the draft model `drafter` proposes `delta` tokens
 * greedily, one single-row forward each (step 3(a)).  Either draft is verified by one target
 * block and the longest agreeing prefix plus one extra token is emitted (step 3(b); Sec. 3.2);
 * the target's cache and, after a drafted step, the draft model's cache are rolled back to the
 * accepted prefix (step 3(c)).  Copy steps do not touch the draft model: before it next
 * drafts it runs over the accepted tokens it has not seen, in blocks of its k_max + 1 rows.
 *   target, drafter: two contexts (different objects) with the same vocabulary;
 *            k, delta <= target's k_max.  Neither may have a cs_loop_begin session open
 *            (the loop buffers of both workspaces serve as scratch).
 *   hist int32 [stride] device, hist_len int32 [1] device, in/out as in cs_decode_loop.
 *   kv_target / kv_len_target [1]: the target's cache, kv_len_target = hist_len - 1 on entry.
 *   kv_drafter / kv_len_drafter [1]: the draft model's cache, holding any prefix
 *            (0 <= kv_len_drafter <= hist_len - 1) of the same history; on return it holds
 *            the positions below the returned kv_len_drafter.
 *   delta = 0: drafter, kv_drafter, kv_len_drafter may be NULL; the loop is then
 *            cs_decode_loop's, driven from the host.
 *   script int32 [max_new] device or NULL: scripted-target mode as in cs_decode_loop.
 *   stats_out host or NULL: attempts / accepted / tau_hist count copy attempts only, no_match
 *            counts every step without a match.  draft_stats_out host uint64 [2] or NULL:
 *            steps the draft model drafted, and its proposals that were accepted.
 * The host reads the match position and the accepted block every step (one or two stream
 * synchronisations per step).  Requires stride >= hist_len + max_new, target max_seq >=
 * hist_len + max_new + max(k, delta), drafter max_seq >= hist_len + max_new + delta
 * (CS_ERR_CAPACITY before anything is launched).  Returns the first error among the host
 * checks, CUDA and the two device status words. */
cs_status cs_decode_loop_drafted(cs_ctx* target, cs_ctx* drafter, int32_t* hist, int32_t* hist_len,
                                 int stride, void* kv_target, int32_t* kv_len_target,
                                 void* kv_drafter, int32_t* kv_len_drafter, int gamma, int k,
                                 int delta, cs_match_policy policy, int max_new, int eos_id,
                                 const int32_t* script, cs_stats* stats_out,
                                 uint64_t* draft_stats_out, void* stream);

/* Measurement aid (no counterpart in the paper): a timeline of the step's kernels taken inside
 * the running pipeline.  `stamps` is a caller-allocated DEVICE array of `capacity` 64-bit slots
 * (zero it once); NULL or capacity 0 switches the aid off.  While it is set, stamped launch i
 * of every step the context enqueues or captures afterwards - search (the scan), block set-up,
 * embedding + first norm, the projection GEMMs, the attention and merge kernels, the LM-head
 * GEMM, acceptance, commit - has each of its CTAs leave the nanosecond time (%globaltimer) at
 * which it finished in stamps[i], largest wins, so stamps[i] - stamps[i-1] is what kernel i added
 * to the pipelined step (the index kernels of cs_set_match_index are not stamped: they count
 * towards the slot that follows).  Set it before cs_loop_begin / the first cs_step_host; it cannot change while a loop
 * is in progress.  cs_stamp_layout returns the number of slots one step uses and writes the
 * kernel family of each slot to the HOST array `family` (0 = layer projection GEMM,
 * 1 = attention, 2 = LM-head GEMM with fused argmax, 3 = merge of the attention's key slices,
 * 4 = everything else).  Costs one atomic per CTA while set, nothing otherwise. */
cs_status cs_set_stamps(cs_ctx* ctx, unsigned long long* stamps, int capacity);
int cs_stamp_layout(const cs_ctx* ctx, int* family, int capacity);

/* Helper off the hot path: computes the KV cache of positions [0, hist_len[b] - 1) by
 * running the forward over the history in blocks with every row forced (no LM head, no
 * acceptance), and sets kv_len[b] = hist_len[b] - 1.  `max_len` (host) is an upper bound
 * of hist_len.  Async. */
cs_status cs_prefill(cs_ctx* ctx, const int32_t* hist, const int32_t* hist_len, int B,
                     int stride, int max_len, void* kv_cache, int32_t* kv_len, void* stream);

/* Building block of the forward of Sec. 3.2, exposed for testing the tensor-core path in
 * isolation: Y[rows][N] (fp32) = X[rows][K] (bf16) times W[N][K]^T (bf16), fp32
 * accumulation.  rows <= 256; K a multiple of 8; X must be readable for
 * ceil(rows/16)*16 rows.  Async. */
cs_status cs_linear(cs_ctx* ctx, const void* X, const void* W, int rows, int N, int K,
                    float* Y, void* stream);

/* Test hook for the bounded waits (no counterpart in the paper): the next cs_linear / GEMM
 * launch of this context leaves out the loads of 64-wide K block `k_block` of every CTA, so the
 * consumer's wait for that block runs out after the context's wait limit (CS_WAIT_LIMIT_US),
 * the CTA drains its other copies, frees its tensor memory and returns, and cs_sync_status
 * reports CS_ERR_TIMEOUT.  Nothing faults and the context stays usable.  Meant for
 * non-clustered launches (a GEMM small enough to run without split-K).  k_block < 0 clears it. */
cs_status cs_debug_drop_tile(cs_ctx* ctx, int k_block);

/* The LM-head stage of the verification forward on its own (Sec. 3.2; App. B.2: greedy
 * token at temperature 0): ids[r] = the lowest token id with the largest logit of
 * X[r] . lm_head^T, for rows already normalised and rounded to bf16.  X bf16 [rows][d_model],
 * readable for ceil(rows/16)*16 rows; ids int32 [rows]; logits_dbg fp32 [rows][vocab] or
 * NULL.  Uses the context's workspace for the per-tile maxima, so it must not overlap other
 * work of the context.  rows <= 256.  Async. */
cs_status cs_lm_head(cs_ctx* ctx, const void* X, int rows, int32_t* ids, float* logits_dbg,
                     void* stream);

/* cs_lm_head for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a deployment convenience, not a step of the method).
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside another framework's
 * allocator or stream callback, in a plug-in that is handed input and output buffers but
 * owns no allocator, or in a process whose device memory is already fully committed.  Such
 * a caller cannot provide the workspace cs_create asks for.  This call needs no context and
 * no workspace: the per-tile (max logit, token id) pairs it needs between the GEMM and the
 * final reduction live in a fixed 512 KB array inside the library image, which every GPU
 * that loads the library holds until the process exits.  It calls no allocating routine.
 *
 *   X bf16 [rows][d_model] (readable for ceil(rows/16)*16 rows), W bf16 [vocab][d_model]
 *   (the LM head), both 16-byte aligned; ids int32 [rows]: the lowest token id with the
 *   largest logit of X[r] . W^T.  d_model a multiple of 8.  Async on `stream`.
 *   Limits: rows <= 64 and vocab <= 131072; anything larger returns CS_ERR_LIMIT and does
 *   nothing.  Other errors, all found before anything is enqueued: CS_ERR_ARG (NULL, sizes,
 *   alignment), CS_ERR_CUDA (no device address for the array, or the driver cannot encode
 *   the operand maps).  A row whose GEMM gave up on a bounded wait gets id -2.
 *
 * The first call on a device looks up the array's device address (and raises the kernel's
 * shared-memory limit); make that first call outside any stream capture, and from one thread
 * (two threads making the first call on the same device at once would both do the set-up).
 * All calls share
 * the one array, which keeps the previous call's contents (only its status word is cleared
 * per call): two calls that overlap on the GPU - different streams, or threads - race on it
 * and give wrong tokens.  Keep calls on one stream, or order them yourself. */
cs_status cs_lm_head_static(const void* X, const void* W, int rows, int vocab, int d_model,
                            int32_t* ids, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* COPYSPEC_H */
