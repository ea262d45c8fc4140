// Shared declarations of the copy-and-verify library: context layout, launch helpers,
// the device status word.  Every .cu file of the library includes this.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "copyspec.h"

// ---------------------------------------------------------------- device status word
// Bits OR-ed into the context's status word by kernels; cs_sync_status maps them.
enum : int {
  CS_DEV_CAPACITY = 1,  // KV cache / history row too small for this step
  CS_DEV_BADARG = 2,    // cs_kv_truncate asked to grow
  CS_DEV_TIMEOUT = 4,   // a bounded wait ran out
  CS_DEV_SMEM = 8       // a kernel found its shared-memory window laid out in a way it cannot use
};

static constexpr int CS_MAX_ROWS = 256;   // rows of one verification block (UMMA N limit)
static constexpr int CS_GEMM_BM = 128;    // out-features per CTA tile (UMMA M)
static constexpr int CS_GEMM_BK = 64;     // K elements per stage (one 128-byte swizzle row)
static constexpr int CS_MAX_GAMMA = 8;
static constexpr int CS_MAX_SPLITS = 8;   // split-K factor limit (portable cluster size)
static constexpr int CS_SPLIT_TILE_CAP = 640;  // tiles * splits never exceeds this (unless splits == 1)

struct GemmPlan {
  CUtensorMap tmW;      // weights [N][K], box 128 x 64, 128-byte swizzle
  const __nv_bfloat16* W;
  int N, K;
  int splits;           // split-K factor
  int kb_per_split;     // 64-wide K blocks per split
  bool allow_split;
};

// how one GEMM is launched for a given block height
struct GemmShape {
  int n_tok;            // token rows rounded up to 16 (UMMA N)
  int mt;               // 128-feature sub-tiles per CTA
  int splits, kb_per_split, stages, stage_bytes, smem;
};

struct LayerPlan {
  GemmPlan qkv, o, gate_up, down;
  const __nv_bfloat16 *attn_norm, *ffn_norm;
};

// device-resident generation loop between cs_loop_begin and cs_loop_end
struct LoopState {
  bool active, use_graph;
  bool use_index;    // the search is the gamma-gram index's lookup instead of the scan
  int32_t *hist, *hist_len, *kv_len;
  const int32_t* script;
  void* kv_cache;
  int B, stride, gamma, k, policy, max_new, eos_id;
  int graph_nodes;   // kernel launches in one step
  cudaGraph_t graph;
  cudaGraphExec_t exec;
  // several steps in one graph: consecutive graph launches leave a gap of some 10 us between them
  cudaGraph_t graph_n;
  cudaGraphExec_t exec_n;
};
static constexpr int CS_LOOP_UNROLL = 4;   // steps per launch of graph_n

// cs_step_host keeps the graph of its last launch shape: the kernels of one step between the
// host -> device and device -> host copies
struct HostStepGraph {
  const void *hist_dev, *hist_len_dev, *kv_cache, *kv_len;
  int B, stride, gamma, k, policy, scripted;
  cudaGraph_t graph;
  cudaGraphExec_t exec;
  // what the device copy of the histories holds: rows [0, uploaded[b]) of up_host -> up_dev
  const void *up_host, *up_dev;
  int up_B, up_stride;
  int uploaded[CS_MAX_ROWS];    // tokens of row b on the device
  int host_len[CS_MAX_ROWS];    // hist_len_host[b] as the previous call left it
};

// cs_verify_step_cached keeps the graphs of its last few launch shapes
struct VerifyGraph {
  const void* key[9];   // last_tok, draft, draft_len, kv_cache, kv_len, script, accept_len, out_tokens, argmax_ids
  int B, k;
  cudaGraph_t graph;
  cudaGraphExec_t exec;
};
static constexpr int CS_VERIFY_GRAPHS = 8;

// Step timeline (cs_set_stamps): every stamped launch of a step owns one 64-bit slot of a
// caller-provided device buffer, into which each of its CTAs leaves the time at which it
// finished (largest wins).  Kernel i's share of the pipelined step is then
// end[i] - end[i - 1], measured inside the running pipeline with no event between launches.
static constexpr int CS_STAMP_MAX = 4096;
enum : int { CS_FAM_GEMM = 0, CS_FAM_ATTENTION = 1, CS_FAM_LMHEAD = 2, CS_FAM_MERGE = 3, CS_FAM_OTHER = 4 };

struct cs_ctx {
  cs_model_config cfg;
  int max_rows;      // max_batch * (k_max + 1)
  int rows_pad;      // rounded up to 16
  int attn_splits;   // split-KV factor
  int num_sms;
  cudaStream_t cap_stream;   // used only to capture the loop's step graph

  const __nv_bfloat16 *embed, *final_norm;
  LayerPlan* layers;  // host array
  GemmPlan lm;

  // workspace partition (device)
  char* ws;
  size_t ws_bytes;
  float* x;                  // residual stream fp32 [rows_pad][d]
  // GEMM / attention operands as two bf16 terms: rows [0, 256) = hi, rows [256, 512) = lo
  __nv_bfloat16* xn;         // normed activations [2*rows_pad][d]
  __nv_bfloat16* attn_out;   // attention output [2*rows_pad][H*Dh]
  __nv_bfloat16* act;        // SwiGLU output [2*rows_pad][F]
  __nv_bfloat16* qbuf;       // rotated queries [2*rows_pad][H*Dh]
  float* qkv;                // QKV projection output fp32 [rows][(H+2Hkv)*Dh]; scratch of cs_linear
  size_t qkv_elems;
  float* attn_o;             // split-KV partial outputs [splits][rows][H][Dh]
  float* attn_ml;            // split-KV (max, sum) [splits][rows][H][2]
  float* ssq;                // sum-of-squares slots of the folded RMSNorm [rows][ssq_stride]
  int ssq_stride;
  float* rope_cs;            // cos/sin of this block [rows][Dh/2][2]
  double* inv_freq;          // theta^(-2i/Dh) [Dh/2]
  float* tile_max;           // LM-head tile maxima [rows_pad][tiles]
  int* tile_idx;             // and their token ids
  int* row_tok;              // token id per row [rows_pad]
  int* row_pos;              // absolute position per row
  int* row_lim;              // number of keys a row attends to (0 = dead row)
  int* row_write;            // 1 = this row's K/V go into the cache
  int* seq_ok;               // per sequence: 1 = takes part in this step
  int* d_status;             // device status word
  // loop state, all [max_batch] unless noted
  int* loop_last;
  int* loop_draft;           // [max_batch][k_max]
  int* loop_dlen;
  int* loop_mpos;
  int* loop_emitted;
  int* loop_done;            // [max_batch] + 1 (last = number of finished sequences)
  int* loop_accept;
  int* loop_out;             // [max_batch][k_max+1]
  int* loop_argmax;          // [max_batch][k_max+1]
  unsigned long long* loop_stats;  // image of cs_stats

  // activation operand maps, rebuilt when the block height changes
  int act_ntok;
  CUtensorMap tmXn, tmAttn, tmAct;

  // tensor-core attention: maps over the whole KV cache (rebuilt when the cache pointer
  // changes) and over the rotated queries (rebuilt when the block height changes)
  CUtensorMap tmKV, tmQ;
  const void* tmKV_base;
  int tmQ_R;
  // Cached lengths [max_batch] that stay as they are until the forward being enqueued has
  // finished, and whose cache rows are complete: set only where the step opens with an
  // ordinary stream-ordered launch (the generation loop); NULL elsewhere.  The attention
  // kernel may then fetch tiles of cached keys before it waits for the preceding kernel.
  const int* kv_len_early;
  // shared-memory opt-ins already made for this context's device (per context, not per
  // process: another context may live on another GPU)
  bool gemm_attr_set;
  int tall_clusters[3][CS_MAX_SPLITS + 1];   // clusters of a tall GEMM launch that can run at once, by sub-tile count and cluster size (0 = not asked yet)
  unsigned attn_mma_attr_set;   // bit DH/32 per head size
  size_t attn_tc_smem_set, attn_tcw_smem_set;
  int attn_force;            // 0 = choose by shape, 1 = mma.sync kernel, 2 = tcgen05 kernel (query rows as M), 3 = tcgen05 kernel (keys as M)
  bool one_term;             // the forward being enqueued feeds its GEMMs the leading bf16 term only
  bool no_graph;             // CS_NO_GRAPH=1 at creation: steps are enqueued kernel by kernel
  unsigned long long wait_limit_ns;   // limit of the kernels' bounded waits (CS_WAIT_LIMIT_US at creation; 2 s)
  int debug_drop_kb;         // test hook: the next GEMM launch leaves out this K block's loads (-1 = none)

  void* match_index;         // cs_set_match_index: the loop searches through this gamma-gram index (NULL = scan)
  int match_index_cap;

  LoopState loop;
  HostStepGraph host_step;
  VerifyGraph verify_graphs[CS_VERIFY_GRAPHS];
  int verify_graph_next;
  unsigned long long* stamp_buf;   // device, caller-owned; NULL = no stamps
  int stamp_cap, stamp_n;          // slots available / handed out for the step being enqueued
  unsigned char stamp_fam[CS_STAMP_MAX];

  char err[256];
};

#define CS_CUDA_OK(ctx, call)                                                          \
  do {                                                                                 \
    cudaError_t e__ = (call);                                                          \
    if (e__ != cudaSuccess) {                                                          \
      if (ctx) snprintf((ctx)->err, sizeof((ctx)->err), "%s: %s", #call,               \
                        cudaGetErrorString(e__));                                      \
      return CS_ERR_CUDA;                                                              \
    }                                                                                  \
  } while (0)

static inline int cs_ceil_div(int a, int b) { return (a + b - 1) / b; }

// slot of the next stamped launch of the step being enqueued (NULL when stamps are off)
static inline unsigned long long* cs_next_stamp(cs_ctx* ctx, int family) {
  if (ctx->stamp_buf == nullptr || ctx->stamp_n >= ctx->stamp_cap || ctx->stamp_n >= CS_STAMP_MAX) return nullptr;
  ctx->stamp_fam[ctx->stamp_n] = (unsigned char)family;
  return ctx->stamp_buf + ctx->stamp_n++;
}
#ifdef __CUDACC__
// called by one thread of a CTA once the CTA's work is done
__device__ __forceinline__ void cs_stamp_end(unsigned long long* slot) {
  if (slot != nullptr) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    atomicMax(slot, t);
  }
}
#endif

// GEMM epilogues
enum : int { CS_EPI_STORE = 0, CS_EPI_ARGMAX = 1, CS_EPI_RESIDUAL = 2, CS_EPI_SWIGLU = 3, CS_EPI_QKV = 4 };

// destination of the QKV epilogue
struct QkvEpi {
  const float* rope_cs;
  const int* row_pos;
  const int* row_write;
  __nv_bfloat16* qbuf;
  __nv_bfloat16* kv;
  int R, layer, H, Hkv, Dh, max_batch, max_seq;
};

// RMSNorm folded into the GEMMs on either side of it.  A residual GEMM that feeds a norm
// (`gain_out` set) also writes gain * x_new as the next GEMM's two-term bf16 operand and, per
// (tile, split-K rank) slot, the sum of squares of the features it finished; the GEMM that
// consumes the norm (`ssq_in` set) adds the slots up in a fixed order and scales its
// accumulators by rsqrt(sum / d + eps), which commutes with the contraction.
struct NormFuse {
  const float* ssq_in;            // [rows][slot_stride], NULL = operand already normalised
  int slots_in, slot_stride;
  float inv_d, eps;
  const __nv_bfloat16* gain_out;  // NULL = no norm follows
  __nv_bfloat16* xn_out;          // [2 * CS_MAX_ROWS][N]: leading terms, then second terms
  float* ssq_out;
};

// Programmatic dependent launch: every kernel of the library lets its successor start
// early and waits for its predecessor before it touches global memory the predecessor
// (or, transitively, anything earlier in the stream) may still be using.
#define CS_PDL_PROLOGUE()                                              \
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     \
  asm volatile("griddepcontrol.wait;" ::: "memory")

template <typename... KArgs, typename... Args>
static inline cudaError_t cs_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                        cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}

// split-K factor limit for a GEMM of `tiles` 128-row tiles and `kb` 64-wide K blocks
static inline int cs_max_splits(int tiles, int kb) {
  int s = CS_SPLIT_TILE_CAP / tiles;
  if (s > CS_MAX_SPLITS) s = CS_MAX_SPLITS;
  if (s > kb / 4) s = kb / 4;
  return s < 1 ? 1 : s;
}

// ------------------------------------------------------------------ kernel launchers
// cs_match.cu
cs_status cs_launch_find_match(const int32_t* hist, const int32_t* hist_len, int B, int stride,
                               int gamma, int k, int policy, int32_t* match_pos, int32_t* draft,
                               int32_t* draft_len, int32_t* last_tok, const int32_t* skip,
                               cudaStream_t st, unsigned long long* stamp = nullptr);
// cs_index.cu
cs_status cs_launch_gram_lookup(const void* index, int B, int capacity_tokens, const int32_t* hist, const int32_t* hist_len,
                                int stride, int gamma, int k, int policy, int32_t* match_pos, int32_t* draft,
                                int32_t* draft_len, int32_t* last_tok, const int32_t* skip, cudaStream_t st);
// inserts the grams that became admissible; overflow is flagged in `status` (NULL = the index's own word)
cs_status cs_launch_gram_update(void* index, int B, int capacity_tokens, const int32_t* hist, const int32_t* hist_len,
                                int stride, int gamma, int max_chunks, int* status, cudaStream_t st);
// cs_gemm.cu
cs_status cs_gemm_plan(cs_ctx* ctx, GemmPlan* g, const void* w, int N, int K, bool allow_split);
cs_status cs_gemm_shape(const cs_ctx* ctx, const GemmPlan* g, int rows, bool two_terms, GemmShape* out);
cs_status cs_make_act_map(cs_ctx* ctx, CUtensorMap* tm, const void* base, int rows_total, int K,
                          int box_rows);
// mode = CS_EPI_*: `out` is the fp32 destination (STORE, RESIDUAL) or the optional logits dump
// (ARGMAX); `act`/F the bf16 destination of SWIGLU
// lo_row: row coordinate (in tmX) of the activation operand's second bf16 term, -1 if X is plain bf16
cs_status cs_launch_gemm(cs_ctx* ctx, const GemmPlan* g, const CUtensorMap* tmX, int lo_row, int rows, int mode,
                         float* out, __nv_bfloat16* act, __nv_bfloat16* act_lo, int F, const QkvEpi* q, const NormFuse* nf,
                         cudaStream_t st);
// cs_layers.cu
void cs_launch_block_setup(cs_ctx* ctx, const int32_t* last_tok, const int32_t* draft,
                           const int32_t* draft_len, const int32_t* kv_len, const int32_t* skip,
                           int B, int k, cudaStream_t st);
void cs_launch_prefill_setup(cs_ctx* ctx, const int32_t* hist, const int32_t* hist_len, int B,
                             int stride, int start, int R, cudaStream_t st);
void cs_launch_embed_rmsnorm(cs_ctx* ctx, const __nv_bfloat16* gain, int rows, cudaStream_t st);
// cs_verify_step replayed from a graph kept per launch shape (all pointers and B, k equal):
// for host-ordered loops that call it with a few fixed sets of buffers.  The launch is one
// stream-ordered unit, so the attention kernel may fetch cached tiles early.
cs_status cs_verify_step_cached(cs_ctx* ctx, const int32_t* last_tok, const int32_t* draft, const int32_t* draft_len,
                                int B, int k, void* kv_cache, int32_t* kv_len, const int32_t* target_script,
                                int32_t* accept_len, int32_t* out_tokens, int32_t* argmax_ids, cudaStream_t st);

void cs_launch_attention(cs_ctx* ctx, const void* kv_cache, int layer, int B, int R,
                         cudaStream_t st);
void cs_launch_attn_merge(cs_ctx* ctx, int nsplit, int rows, cudaStream_t st);
// tcgen05 path (head_dim 128, at most 128 query heads per KV head); returns the number of key
// slices written, 0 when the shape is not covered, -1 on a host error (ctx->err set)
int cs_launch_attention_tc(cs_ctx* ctx, const void* kv_cache, int layer, int B, int R, cudaStream_t st);
// the same contract, keys and head dims as the M dimension (long key ranges); `probe` only answers
// how many key tiles a CTA of the query-rows-as-M kernel would walk at most
int cs_launch_attention_tcw(cs_ctx* ctx, const void* kv_cache, int layer, int B, int R, cudaStream_t st);
int cs_attention_tc_tiles_per_cta(const cs_ctx* ctx, int B, int R);
// bf16 tensor map of rank <= 5, 128-byte swizzle; dims/box innermost first, strides for dims 1..
cs_status cs_encode_tiled(cs_ctx* ctx, CUtensorMap* tm, const void* base, int rank, const unsigned long long* dims,
                          const unsigned long long* strides_bytes, const unsigned* box);
void cs_launch_accept(cs_ctx* ctx, int B, int k, const int32_t* draft, const int32_t* draft_len,
                      const int32_t* script, int script_stride, const int32_t* script_off,
                      int script_limit, int32_t* accept_len, int32_t* out_tokens,
                      int32_t* argmax_ids, int32_t* kv_len, int update_kv, cudaStream_t st);
void cs_launch_tile_reduce(cs_ctx* ctx, int rows, int32_t* ids, cudaStream_t st);
void cs_launch_truncate(cs_ctx* ctx, int32_t* kv_len, const int32_t* new_len, int B,
                        cudaStream_t st);
void cs_launch_prefill_finish(cs_ctx* ctx, const int32_t* hist_len, int32_t* kv_len, int B,
                              cudaStream_t st);
void cs_launch_loop_init(cs_ctx* ctx, const int32_t* hist_len, const int32_t* kv_len, int B,
                         int stride, int max_new, int k, cudaStream_t st);
void cs_launch_loop_commit(cs_ctx* ctx, int32_t* hist, int32_t* hist_len, int B, int stride,
                           int32_t* kv_len, int k, int max_new, int eos_id, int scripted,
                           cudaStream_t st);
