// C ABI of the copy-and-verify library: argument checks, workspace layout, the chain of
// kernels of one verification step and the device-resident generation loop.
#include <math.h>
#include <stdlib.h>

#include <new>

#include <string.h>

#include "cs_common.cuh"

namespace {

struct WsLayout {
  size_t x, xn, attn_out, act, qbuf, partial, attn_o, attn_ml, ssq, rope_cs, inv_freq, tile_max, tile_idx,
      row_tok, row_pos, row_lim, row_write, seq_ok, status, loop_last, loop_draft, loop_dlen, loop_mpos,
      loop_emitted, loop_done, loop_accept, loop_out, loop_argmax, loop_stats, total;
  size_t qkv_elems;
  int attn_splits;
};

bool config_ok(const cs_model_config* c) {
  if (c == nullptr) return false;
  if (c->n_layers < 1 || c->d_model < 8 || c->n_heads < 1 || c->n_kv_heads < 1 || c->d_ffn < 8 ||
      c->vocab < 1 || c->max_seq < 1 || c->max_batch < 1 || c->k_max < 0)
    return false;
  if (c->head_dim != 32 && c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->n_heads % c->n_kv_heads) return false;
  if ((long)c->max_batch * (c->k_max + 1) > CS_MAX_ROWS) return false;
  if (c->d_model % 8 || c->d_ffn % 8 || (c->n_heads * c->head_dim) % 8) return false;
  return true;
}

size_t take(size_t* off, size_t bytes) {
  const size_t at = *off;
  *off = (at + bytes + 1023) & ~(size_t)1023;
  return at;
}

WsLayout ws_layout(const cs_model_config* c) {
  WsLayout L;
  const size_t rows = CS_MAX_ROWS;
  const size_t d = c->d_model, qd = (size_t)c->n_heads * c->head_dim, F = c->d_ffn;
  const size_t qkv = qd + 2 * (size_t)c->n_kv_heads * c->head_dim;
  L.qkv_elems = rows * (qkv > 4096 ? qkv : 4096);
  int as = cs_ceil_div(c->max_seq, 128);
  L.attn_splits = as < 1 ? 1 : (as > 64 ? 64 : as);
  const size_t lm_tiles = cs_ceil_div(c->vocab, CS_GEMM_BM);
  size_t off = 0;
  L.x = take(&off, rows * d * 4);
  // operands carried as two bf16 terms: hi rows then lo rows
  L.xn = take(&off, 2 * rows * d * 2);
  L.attn_out = take(&off, 2 * rows * qd * 2);
  L.act = take(&off, 2 * rows * F * 2);
  L.qbuf = take(&off, 2 * rows * qd * 2);
  L.partial = take(&off, L.qkv_elems * 4);
  L.attn_o = take(&off, (size_t)L.attn_splits * rows * qd * 4);
  L.attn_ml = take(&off, (size_t)L.attn_splits * rows * c->n_heads * 2 * 4);
  L.ssq = take(&off, rows * (size_t)cs_ceil_div(c->d_model, CS_GEMM_BM) * CS_MAX_SPLITS * 4);
  L.rope_cs = take(&off, rows * c->head_dim * 4);
  L.inv_freq = take(&off, (size_t)c->head_dim / 2 * 8);
  L.tile_max = take(&off, lm_tiles * rows * 4);
  L.tile_idx = take(&off, lm_tiles * rows * 4);
  L.row_tok = take(&off, rows * 4);
  L.row_pos = take(&off, rows * 4);
  L.row_lim = take(&off, rows * 4);
  L.row_write = take(&off, rows * 4);
  L.seq_ok = take(&off, rows * 4);
  L.status = take(&off, 256);
  L.loop_last = take(&off, rows * 4);
  L.loop_draft = take(&off, rows * 4);
  L.loop_dlen = take(&off, rows * 4);
  L.loop_mpos = take(&off, rows * 4);
  L.loop_emitted = take(&off, rows * 4);
  L.loop_done = take(&off, (rows + 1) * 4);
  L.loop_accept = take(&off, rows * 4);
  L.loop_out = take(&off, rows * 4);
  L.loop_argmax = take(&off, rows * 4);
  L.loop_stats = take(&off, sizeof(cs_stats));
  L.total = off;
  return L;
}

// cs_create has no context to leave an error text in: the last failure of this thread is kept here
thread_local char g_create_err[256] = "";

cs_status fail(cs_ctx* ctx, cs_status s, const char* msg) {
  if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s", msg);
  return s;
}

cs_status ensure_act_maps(cs_ctx* ctx, int n_tok) {
  if (ctx->act_ntok == n_tok) return CS_OK;
  const cs_model_config& c = ctx->cfg;
  cs_status s;
  if ((s = cs_make_act_map(ctx, &ctx->tmXn, ctx->xn, 2 * CS_MAX_ROWS, c.d_model, n_tok)) != CS_OK) return s;
  if ((s = cs_make_act_map(ctx, &ctx->tmAttn, ctx->attn_out, 2 * CS_MAX_ROWS, c.n_heads * c.head_dim, n_tok)) != CS_OK)
    return s;
  if ((s = cs_make_act_map(ctx, &ctx->tmAct, ctx->act, 2 * CS_MAX_ROWS, c.d_ffn, n_tok)) != CS_OK) return s;
  ctx->act_ntok = n_tok;
  return CS_OK;
}

// The forward of Sec. 3.2 over the rows prepared by a *_setup kernel: B sequences of R
// rows each.  With `with_lm` the LM head leaves per-tile (max, id) pairs for k_accept.
cs_status enqueue_forward(cs_ctx* ctx, int B, int R, void* kv_cache, bool with_lm, float* logits,
                          cudaStream_t st) {
  const cs_model_config& c = ctx->cfg;
  const int rows = B * R;
  // second bf16 term of every activation operand (row offset in the operand maps), or -1 when the
  // caller settles for the leading term
  const int lo_row = ctx->one_term ? -1 : CS_MAX_ROWS;
  cs_status s = ensure_act_maps(ctx, cs_ceil_div(rows, 16) * 16);
  if (s != CS_OK) return s;
  // Only the first RMSNorm runs as a kernel.  Every later one is folded into the GEMMs around
  // it: the residual GEMM before it writes gain * x (two bf16 terms) and sums of squares, the
  // GEMM after it scales its accumulators by 1/rms.
  NormFuse take_norm = {};           // how the next norm-consuming GEMM finds its 1/rms
  for (int l = 0; l < c.n_layers; ++l) {
    const LayerPlan& L = ctx->layers[l];
    if (l == 0) {
      cs_launch_embed_rmsnorm(ctx, L.attn_norm, rows, st);
    }
    const QkvEpi qe = {ctx->rope_cs, ctx->row_pos, ctx->row_write, ctx->qbuf, static_cast<__nv_bfloat16*>(kv_cache),
                       R, l, c.n_heads, c.n_kv_heads, c.head_dim, c.max_batch, c.max_seq};
    s = cs_launch_gemm(ctx, &L.qkv, &ctx->tmXn, lo_row, rows, CS_EPI_QKV, nullptr, nullptr, nullptr, 0, &qe,
                       &take_norm, st);
    if (s != CS_OK) return s;
    cs_launch_attention(ctx, kv_cache, l, B, R, st);
    NormFuse give = {};
    give.gain_out = L.ffn_norm;
    give.xn_out = ctx->xn;
    give.ssq_out = ctx->ssq;
    give.slot_stride = ctx->ssq_stride;
    s = cs_launch_gemm(ctx, &L.o, &ctx->tmAttn, lo_row, rows, CS_EPI_RESIDUAL, ctx->x, nullptr, nullptr, 0, nullptr,
                       &give, st);
    if (s != CS_OK) return s;
    take_norm = NormFuse{};
    take_norm.ssq_in = ctx->ssq;
    {
      GemmShape sh;
      if (cs_gemm_shape(ctx, &L.o, rows, lo_row >= 0, &sh) != CS_OK) return fail(ctx, CS_ERR_UNSUPPORTED, "no launch shape for the attention-output GEMM");
      take_norm.slots_in = cs_ceil_div(L.o.N, CS_GEMM_BM) * sh.splits;
    }
    take_norm.slot_stride = ctx->ssq_stride;
    take_norm.inv_d = 1.f / (float)c.d_model;
    take_norm.eps = c.rms_eps;
    s = cs_launch_gemm(ctx, &L.gate_up, &ctx->tmXn, lo_row, rows, CS_EPI_SWIGLU, nullptr, ctx->act,
                       ctx->act + (size_t)CS_MAX_ROWS * c.d_ffn, c.d_ffn, nullptr, &take_norm, st);
    if (s != CS_OK) return s;
    // the norm after this layer: the next layer's, or the final one before the LM head
    const __nv_bfloat16* next_gain = (l + 1 < c.n_layers) ? ctx->layers[l + 1].attn_norm : (with_lm ? ctx->final_norm : nullptr);
    give.gain_out = next_gain;
    s = cs_launch_gemm(ctx, &L.down, &ctx->tmAct, lo_row, rows, CS_EPI_RESIDUAL, ctx->x, nullptr, nullptr, 0, nullptr,
                       &give, st);
    if (s != CS_OK) return s;
    {
      GemmShape sh;
      if (cs_gemm_shape(ctx, &L.down, rows, lo_row >= 0, &sh) != CS_OK) return fail(ctx, CS_ERR_UNSUPPORTED, "no launch shape for the down GEMM");
      take_norm.slots_in = cs_ceil_div(L.down.N, CS_GEMM_BM) * sh.splits;
    }
  }
  if (with_lm) {
    s = cs_launch_gemm(ctx, &ctx->lm, &ctx->tmXn, lo_row, rows, CS_EPI_ARGMAX, logits, nullptr, nullptr, 0, nullptr,
                       &take_norm, st);
    if (s != CS_OK) return s;
  }
  CS_CUDA_OK(ctx, cudaGetLastError());
  return CS_OK;
}

// One iteration of the generation loop (App. B.3 steps 1, 2, 4) on device-resident state.
cs_status enqueue_loop_step(cs_ctx* ctx, cudaStream_t st) {
  const LoopState& L = ctx->loop;
  ctx->stamp_n = 0;
  // App. B.3 step 1: the scan, or the lookup in the gamma-gram index (Sec. 3.1) - same outputs
  cs_status r = L.use_index
                    ? cs_launch_gram_lookup(ctx->match_index, L.B, ctx->match_index_cap, L.hist, L.hist_len, L.stride, L.gamma,
                                            L.k, L.policy, ctx->loop_mpos, ctx->loop_draft, ctx->loop_dlen, ctx->loop_last,
                                            ctx->loop_done, st)
                    : cs_launch_find_match(L.hist, L.hist_len, L.B, L.stride, L.gamma, L.k, L.policy, ctx->loop_mpos,
                                           ctx->loop_draft, ctx->loop_dlen, ctx->loop_last, ctx->loop_done, st,
                                           cs_next_stamp(ctx, CS_FAM_OTHER));
  if (r != CS_OK) return fail(ctx, r, "match kernel launch failed");
  cs_launch_block_setup(ctx, ctx->loop_last, ctx->loop_draft, ctx->loop_dlen, L.kv_len, ctx->loop_done, L.B, L.k, st);
  // the step opened with a stream-ordered launch and nothing before k_loop_commit changes kv_len
  ctx->kv_len_early = L.kv_len;
  r = enqueue_forward(ctx, L.B, L.k + 1, L.kv_cache, true, nullptr, st);
  ctx->kv_len_early = nullptr;
  if (r != CS_OK) return r;
  cs_launch_accept(ctx, L.B, L.k, ctx->loop_draft, ctx->loop_dlen, L.script, L.max_new, ctx->loop_emitted, L.max_new,
                   ctx->loop_accept, ctx->loop_out, ctx->loop_argmax, L.kv_len, 0, st);
  cs_launch_loop_commit(ctx, L.hist, L.hist_len, L.B, L.stride, L.kv_len, L.k, L.max_new, L.eos_id,
                        L.script != nullptr, st);
  if (L.use_index) {
    // App. B.3 step 2(d): the grams that the appended tokens made admissible enter the index
    r = cs_launch_gram_update(ctx->match_index, L.B, ctx->match_index_cap, L.hist, L.hist_len, L.stride, L.gamma, 1,
                              ctx->d_status, st);
    if (r != CS_OK) return fail(ctx, r, "index update launch failed");
  }
  CS_CUDA_OK(ctx, cudaGetLastError());
  return CS_OK;
}

cs_status status_from_bits(cs_ctx* ctx, int bits) {
  if (bits & CS_DEV_TIMEOUT) return fail(ctx, CS_ERR_TIMEOUT, "a bounded device-side wait ran out");
  if (bits & CS_DEV_CAPACITY) return fail(ctx, CS_ERR_CAPACITY, "KV cache or history row too small for a sequence");
  if (bits & CS_DEV_SMEM) return fail(ctx, CS_ERR_UNSUPPORTED, "attention kernel could not place its barriers in shared memory");
  if (bits & CS_DEV_BADARG) return fail(ctx, CS_ERR_ARG, "device-side argument check failed (lengths inconsistent)");
  return CS_OK;
}

}  // namespace

extern "C" {

size_t cs_workspace_bytes(const cs_model_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return ws_layout(cfg).total;
}

const char* cs_last_error(const cs_ctx* ctx) { return ctx ? ctx->err : g_create_err; }

cs_status cs_create(cs_ctx** out, const cs_model_config* cfg, const cs_weights* w, void* workspace,
                    size_t workspace_bytes) {
  auto create_fail = [](cs_status st, const char* msg) {
    snprintf(g_create_err, sizeof(g_create_err), "cs_create: %s", msg);
    return st;
  };
  if (out == nullptr) return create_fail(CS_ERR_ARG, "NULL output pointer");
  *out = nullptr;
  if (cfg == nullptr || w == nullptr || workspace == nullptr) return create_fail(CS_ERR_ARG, "NULL argument");
  if (!config_ok(cfg)) return create_fail(CS_ERR_SHAPE, "model configuration outside what the kernels support");
  if (w->embed == nullptr || w->lm_head == nullptr || w->final_norm == nullptr || w->attn_norm == nullptr ||
      w->wqkv == nullptr || w->wo == nullptr || w->ffn_norm == nullptr || w->w_gate_up == nullptr ||
      w->w_down == nullptr)
    return create_fail(CS_ERR_ARG, "NULL weight pointer");
  const WsLayout L = ws_layout(cfg);
  if (workspace_bytes < L.total) return create_fail(CS_ERR_CAPACITY, "workspace smaller than cs_workspace_bytes");
  if (reinterpret_cast<uintptr_t>(workspace) & 1023) return create_fail(CS_ERR_ARG, "workspace not 1024-byte aligned");

  cs_ctx* ctx = new (std::nothrow) cs_ctx();
  if (ctx == nullptr) return create_fail(CS_ERR_ARG, "out of host memory");
  memset(static_cast<void*>(ctx), 0, sizeof(*ctx));
  ctx->cfg = *cfg;
  ctx->max_rows = cfg->max_batch * (cfg->k_max + 1);
  ctx->rows_pad = CS_MAX_ROWS;
  ctx->attn_splits = L.attn_splits;
  {
    // the environment switches of the library, all read here and nowhere else
    const char* k = getenv("CS_ATTN_KERNEL");
    ctx->attn_force = (k == nullptr) ? 0 : (strcmp(k, "mma") == 0 ? 1 : (strcmp(k, "tc") == 0 ? 2 : (strcmp(k, "tcw") == 0 ? 3 : 0)));
    const char* ng = getenv("CS_NO_GRAPH");
    ctx->no_graph = ng != nullptr && ng[0] == '1';
    const char* wl = getenv("CS_WAIT_LIMIT_US");
    const long long us = (wl != nullptr) ? atoll(wl) : 0;
    ctx->wait_limit_ns = (us > 0) ? (unsigned long long)us * 1000ull : 2000000000ull;
    ctx->debug_drop_kb = -1;
  }
  ctx->qkv_elems = L.qkv_elems;
  ctx->layers = new (std::nothrow) LayerPlan[cfg->n_layers];
  cs_status s = CS_OK;
  int dev = 0;
  cudaDeviceProp prop;
#define CREATE_OK(call)                                                                        \
  do {                                                                                         \
    cudaError_t e__ = (call);                                                                  \
    if (e__ != cudaSuccess) {                                                                  \
      snprintf(g_create_err, sizeof(g_create_err), "cs_create: %s: %s", #call, cudaGetErrorString(e__)); \
      cs_destroy(ctx);                                                                         \
      return CS_ERR_CUDA;                                                                      \
    }                                                                                          \
  } while (0)
  if (ctx->layers == nullptr) { cs_destroy(ctx); return create_fail(CS_ERR_ARG, "out of host memory"); }
  CREATE_OK(cudaGetDevice(&dev));
  CREATE_OK(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) {
    snprintf(g_create_err, sizeof(g_create_err), "cs_create: this library is built for sm_100a only (device is sm_%d%d)",
             prop.major, prop.minor);
    cs_destroy(ctx);
    return CS_ERR_UNSUPPORTED;
  }
  ctx->num_sms = prop.multiProcessorCount;
  CREATE_OK(cudaStreamCreateWithFlags(&ctx->cap_stream, cudaStreamNonBlocking));
  char* base = static_cast<char*>(workspace);
  ctx->ws = base;
  ctx->ws_bytes = L.total;
  CREATE_OK(cudaMemset(base, 0, L.total));
  ctx->x = reinterpret_cast<float*>(base + L.x);
  ctx->xn = reinterpret_cast<__nv_bfloat16*>(base + L.xn);
  ctx->attn_out = reinterpret_cast<__nv_bfloat16*>(base + L.attn_out);
  ctx->act = reinterpret_cast<__nv_bfloat16*>(base + L.act);
  ctx->qbuf = reinterpret_cast<__nv_bfloat16*>(base + L.qbuf);
  ctx->qkv = reinterpret_cast<float*>(base + L.partial);
  ctx->attn_o = reinterpret_cast<float*>(base + L.attn_o);
  ctx->attn_ml = reinterpret_cast<float*>(base + L.attn_ml);
  ctx->ssq = reinterpret_cast<float*>(base + L.ssq);
  ctx->ssq_stride = cs_ceil_div(ctx->cfg.d_model, CS_GEMM_BM) * CS_MAX_SPLITS;
  ctx->rope_cs = reinterpret_cast<float*>(base + L.rope_cs);
  ctx->inv_freq = reinterpret_cast<double*>(base + L.inv_freq);
  ctx->tile_max = reinterpret_cast<float*>(base + L.tile_max);
  ctx->tile_idx = reinterpret_cast<int*>(base + L.tile_idx);
  ctx->row_tok = reinterpret_cast<int*>(base + L.row_tok);
  ctx->row_pos = reinterpret_cast<int*>(base + L.row_pos);
  ctx->row_lim = reinterpret_cast<int*>(base + L.row_lim);
  ctx->row_write = reinterpret_cast<int*>(base + L.row_write);
  ctx->seq_ok = reinterpret_cast<int*>(base + L.seq_ok);
  ctx->d_status = reinterpret_cast<int*>(base + L.status);
  ctx->loop_last = reinterpret_cast<int*>(base + L.loop_last);
  ctx->loop_draft = reinterpret_cast<int*>(base + L.loop_draft);
  ctx->loop_dlen = reinterpret_cast<int*>(base + L.loop_dlen);
  ctx->loop_mpos = reinterpret_cast<int*>(base + L.loop_mpos);
  ctx->loop_emitted = reinterpret_cast<int*>(base + L.loop_emitted);
  ctx->loop_done = reinterpret_cast<int*>(base + L.loop_done);
  ctx->loop_accept = reinterpret_cast<int*>(base + L.loop_accept);
  ctx->loop_out = reinterpret_cast<int*>(base + L.loop_out);
  ctx->loop_argmax = reinterpret_cast<int*>(base + L.loop_argmax);
  ctx->loop_stats = reinterpret_cast<unsigned long long*>(base + L.loop_stats);

  // rotary frequencies theta^(-2i/Dh), in double
  {
    const int half = cfg->head_dim / 2;
    double f[64];
    for (int i = 0; i < half; ++i) f[i] = pow((double)cfg->rope_theta, -2.0 * i / cfg->head_dim);
    CREATE_OK(cudaMemcpy(ctx->inv_freq, f, sizeof(double) * half, cudaMemcpyHostToDevice));
  }
  ctx->embed = static_cast<const __nv_bfloat16*>(w->embed);
  ctx->final_norm = static_cast<const __nv_bfloat16*>(w->final_norm);
  const int d = cfg->d_model, qd = cfg->n_heads * cfg->head_dim, F = cfg->d_ffn;
  const int qkv = qd + 2 * cfg->n_kv_heads * cfg->head_dim;
  for (int l = 0; l < cfg->n_layers && s == CS_OK; ++l) {
    LayerPlan& P = ctx->layers[l];
    if (!w->attn_norm[l] || !w->wqkv[l] || !w->wo[l] || !w->ffn_norm[l] || !w->w_gate_up[l] || !w->w_down[l]) {
      s = CS_ERR_ARG;
      break;
    }
    P.attn_norm = static_cast<const __nv_bfloat16*>(w->attn_norm[l]);
    P.ffn_norm = static_cast<const __nv_bfloat16*>(w->ffn_norm[l]);
    if ((s = cs_gemm_plan(ctx, &P.qkv, w->wqkv[l], qkv, d, true)) != CS_OK) break;
    if ((s = cs_gemm_plan(ctx, &P.o, w->wo[l], d, qd, true)) != CS_OK) break;
    if ((s = cs_gemm_plan(ctx, &P.gate_up, w->w_gate_up[l], cs_ceil_div(F, 64) * 128, d, true)) != CS_OK) break;
    if ((s = cs_gemm_plan(ctx, &P.down, w->w_down[l], d, F, true)) != CS_OK) break;
  }
  if (s == CS_OK) s = cs_gemm_plan(ctx, &ctx->lm, w->lm_head, cfg->vocab, d, false);
  if (s != CS_OK) {
    snprintf(g_create_err, sizeof(g_create_err), "cs_create: %.200s", ctx->err[0] ? ctx->err : "NULL layer weight pointer");
    cs_destroy(ctx);
    return s;
  }
#undef CREATE_OK
  *out = ctx;
  return CS_OK;
}

void cs_destroy(cs_ctx* ctx) {
  if (ctx == nullptr) return;
  cs_loop_end(ctx);
  if (ctx->cap_stream) cudaStreamDestroy(ctx->cap_stream);
  for (int i = 0; i < CS_VERIFY_GRAPHS; ++i) {
    if (ctx->verify_graphs[i].exec) cudaGraphExecDestroy(ctx->verify_graphs[i].exec);
    if (ctx->verify_graphs[i].graph) cudaGraphDestroy(ctx->verify_graphs[i].graph);
  }
  if (ctx->host_step.exec) cudaGraphExecDestroy(ctx->host_step.exec);
  if (ctx->host_step.graph) cudaGraphDestroy(ctx->host_step.graph);
  delete[] ctx->layers;
  delete ctx;
}

cs_status cs_sync_status(cs_ctx* ctx, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int bits = 0;
  CS_CUDA_OK(ctx, cudaMemcpyAsync(&bits, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  CS_CUDA_OK(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st));
  CS_CUDA_OK(ctx, cudaStreamSynchronize(st));
  return status_from_bits(ctx, bits);
}

cs_status cs_find_match(const int32_t* hist, const int32_t* hist_len, int B, int stride, int gamma, int k,
                        cs_match_policy policy, int32_t* match_pos, int32_t* draft, int32_t* draft_len,
                        void* stream) {
  if (B < 0 || k < 0 || stride < 0) return CS_ERR_ARG;
  if (gamma < 1 || gamma > CS_MAX_GAMMA) return CS_ERR_ARG;
  if (policy != CS_MATCH_LATEST && policy != CS_MATCH_FIRST) return CS_ERR_ARG;
  if (B == 0) return CS_OK;
  if (B > 65535) return CS_ERR_ARG;
  if (hist == nullptr || hist_len == nullptr || match_pos == nullptr || draft_len == nullptr ||
      (draft == nullptr && k > 0))
    return CS_ERR_ARG;
  return cs_launch_find_match(hist, hist_len, B, stride, gamma, k, (int)policy, match_pos, draft, draft_len,
                              nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

cs_status cs_verify_step(cs_ctx* ctx, const int32_t* last_tok, const int32_t* draft, const int32_t* draft_len,
                         int B, int k, void* kv_cache, int32_t* kv_len, const int32_t* target_script,
                         int32_t* accept_len, int32_t* out_tokens, int32_t* argmax_ids, float* logits_dbg,
                         void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (B < 1 || B > ctx->cfg.max_batch || k < 0 || k > ctx->cfg.k_max) return fail(ctx, CS_ERR_ARG, "B or k out of range");
  if (last_tok == nullptr || draft_len == nullptr || (draft == nullptr && k > 0) || kv_cache == nullptr ||
      kv_len == nullptr || accept_len == nullptr || out_tokens == nullptr || argmax_ids == nullptr)
    return fail(ctx, CS_ERR_ARG, "NULL argument");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->stamp_n = 0;
  cs_launch_block_setup(ctx, last_tok, draft, draft_len, kv_len, nullptr, B, k, st);
  cs_status s = enqueue_forward(ctx, B, k + 1, kv_cache, true, logits_dbg, st);
  if (s != CS_OK) return s;
  cs_launch_accept(ctx, B, k, draft, draft_len, target_script, k + 1, nullptr, k + 1, accept_len, out_tokens,
                   argmax_ids, kv_len, 1, st);
  CS_CUDA_OK(ctx, cudaGetLastError());
  return CS_OK;
}

}  // extern "C"

cs_status cs_verify_step_cached(cs_ctx* ctx, const int32_t* last_tok, const int32_t* draft, const int32_t* draft_len,
                                int B, int k, void* kv_cache, int32_t* kv_len, const int32_t* target_script,
                                int32_t* accept_len, int32_t* out_tokens, int32_t* argmax_ids, cudaStream_t st) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (ctx->no_graph)
    return cs_verify_step(ctx, last_tok, draft, draft_len, B, k, kv_cache, kv_len, target_script, accept_len,
                          out_tokens, argmax_ids, nullptr, st);
  if (B < 1 || B > ctx->cfg.max_batch || k < 0 || k > ctx->cfg.k_max) return fail(ctx, CS_ERR_ARG, "B or k out of range");
  if (last_tok == nullptr || draft_len == nullptr || (draft == nullptr && k > 0) || kv_cache == nullptr ||
      kv_len == nullptr || accept_len == nullptr || out_tokens == nullptr || argmax_ids == nullptr)
    return fail(ctx, CS_ERR_ARG, "NULL argument");
  const void* key[9] = {last_tok, draft, draft_len, kv_cache, kv_len, target_script, accept_len, out_tokens, argmax_ids};
  VerifyGraph* g = nullptr;
  for (int i = 0; i < CS_VERIFY_GRAPHS && g == nullptr; ++i) {
    VerifyGraph& c = ctx->verify_graphs[i];
    if (c.exec != nullptr && c.B == B && c.k == k && memcmp(c.key, key, sizeof(key)) == 0) g = &c;
  }
  if (g == nullptr) {
    g = &ctx->verify_graphs[ctx->verify_graph_next];
    ctx->verify_graph_next = (ctx->verify_graph_next + 1) % CS_VERIFY_GRAPHS;
    if (g->exec) cudaGraphExecDestroy(g->exec);
    if (g->graph) cudaGraphDestroy(g->graph);
    *g = VerifyGraph{};
    cs_status s = ensure_act_maps(ctx, cs_ceil_div(B * (k + 1), 16) * 16);   // host work that must precede capture
    if (s != CS_OK) return s;
    CS_CUDA_OK(ctx, cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeRelaxed));
    ctx->stamp_n = 0;
    cs_launch_block_setup(ctx, last_tok, draft, draft_len, kv_len, nullptr, B, k, ctx->cap_stream);
    ctx->kv_len_early = kv_len;      // nothing before the acceptance kernel changes it
    s = enqueue_forward(ctx, B, k + 1, kv_cache, true, nullptr, ctx->cap_stream);
    ctx->kv_len_early = nullptr;
    if (s == CS_OK)
      cs_launch_accept(ctx, B, k, draft, draft_len, target_script, k + 1, nullptr, k + 1, accept_len, out_tokens,
                       argmax_ids, kv_len, 1, ctx->cap_stream);
    cudaError_t e = cudaStreamEndCapture(ctx->cap_stream, &g->graph);
    if (s == CS_OK && e == cudaSuccess) e = cudaGraphInstantiate(&g->exec, g->graph, 0);
    if (s != CS_OK || e != cudaSuccess) {
      if (g->graph) cudaGraphDestroy(g->graph);
      *g = VerifyGraph{};
      if (s != CS_OK) return s;
      CS_CUDA_OK(ctx, e);
    }
    memcpy(g->key, key, sizeof(key));
    g->B = B;
    g->k = k;
  }
  CS_CUDA_OK(ctx, cudaGraphLaunch(g->exec, st));
  return CS_OK;
}

extern "C" {

cs_status cs_step_host(cs_ctx* ctx, int32_t* hist_host, int32_t* hist_len_host, int B, int stride,
                       int32_t* hist_dev, int32_t* hist_len_dev, void* kv_cache, int32_t* kv_len, int gamma, int k,
                       cs_match_policy policy, const int32_t* script_host, int32_t* accept_len_host,
                       int32_t* out_tokens_host, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (B < 1 || B > ctx->cfg.max_batch || k < 0 || k > ctx->cfg.k_max || gamma < 1 || gamma > CS_MAX_GAMMA || stride < 1)
    return fail(ctx, CS_ERR_ARG, "B, k, gamma or stride out of range");
  if (policy != CS_MATCH_LATEST && policy != CS_MATCH_FIRST) return fail(ctx, CS_ERR_ARG, "bad policy");
  if (hist_host == nullptr || hist_len_host == nullptr || hist_dev == nullptr || hist_len_dev == nullptr ||
      kv_cache == nullptr || kv_len == nullptr || accept_len_host == nullptr || out_tokens_host == nullptr)
    return fail(ctx, CS_ERR_ARG, "NULL argument");
  for (int b = 0; b < B; ++b)
    if (hist_len_host[b] < 1 || hist_len_host[b] + k + 1 > stride)
      return fail(ctx, CS_ERR_CAPACITY, "history row too short for one more block");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // ---- host -> device: the tokens the device copy of each history lacks (everything on the first
  // call with these buffers, afterwards what the previous call appended), the lengths, this step's
  // script rows
  HostStepGraph& G = ctx->host_step;
  const bool known = G.up_host == hist_host && G.up_dev == hist_dev && G.up_B == B && G.up_stride == stride;
  for (int b = 0; b < B; ++b) {
    const int n = hist_len_host[b];
    const int have = (known && G.host_len[b] == n && G.uploaded[b] <= n) ? G.uploaded[b] : 0;
    if (n > have)
      CS_CUDA_OK(ctx, cudaMemcpyAsync(hist_dev + (size_t)b * stride + have, hist_host + (size_t)b * stride + have,
                                      (size_t)(n - have) * 4, cudaMemcpyHostToDevice, st));
    G.uploaded[b] = n;
  }
  G.up_host = hist_host; G.up_dev = hist_dev; G.up_B = B; G.up_stride = stride;
  CS_CUDA_OK(ctx, cudaMemcpyAsync(hist_len_dev, hist_len_host, (size_t)B * 4, cudaMemcpyHostToDevice, st));
  const int32_t* script_dev = nullptr;
  if (script_host != nullptr) {
    CS_CUDA_OK(ctx, cudaMemcpyAsync(ctx->loop_emitted, script_host, (size_t)B * (k + 1) * 4, cudaMemcpyHostToDevice, st));
    script_dev = ctx->loop_emitted;
  }
  // ---- App. B.3 step 1 (search, gather), step 2 (verify, accept, truncate): the kernels of one
  // step, replayed as a graph while the launch shape and the buffers stay the same
  // (CS_NO_GRAPH=1 enqueues them one by one)
  const bool use_graph = !ctx->no_graph;
  const bool same = G.exec != nullptr && G.hist_dev == hist_dev && G.hist_len_dev == hist_len_dev &&
                    G.kv_cache == kv_cache && G.kv_len == kv_len && G.B == B && G.stride == stride &&
                    G.gamma == gamma && G.k == k && G.policy == (int)policy && G.scripted == (script_dev != nullptr);
  auto enqueue = [&](cudaStream_t q) -> cs_status {
    ctx->stamp_n = 0;
    cs_status r = cs_launch_find_match(hist_dev, hist_len_dev, B, stride, gamma, k, (int)policy, ctx->loop_mpos,
                                       ctx->loop_draft, ctx->loop_dlen, ctx->loop_last, nullptr, q);
    if (r != CS_OK) return fail(ctx, r, "match kernel launch failed");
    cs_launch_block_setup(ctx, ctx->loop_last, ctx->loop_draft, ctx->loop_dlen, kv_len, nullptr, B, k, q);
    // the search opens the step stream-ordered and every call ends synchronised, so the cached
    // rows and kv_len are settled while the forward runs
    ctx->kv_len_early = kv_len;
    r = enqueue_forward(ctx, B, k + 1, kv_cache, true, nullptr, q);
    ctx->kv_len_early = nullptr;
    if (r != CS_OK) return r;
    cs_launch_accept(ctx, B, k, ctx->loop_draft, ctx->loop_dlen, script_dev, k + 1, nullptr, k + 1, ctx->loop_accept,
                     ctx->loop_out, ctx->loop_argmax, kv_len, 1, q);
    return CS_OK;
  };
  cs_status s = CS_OK;
  if (!use_graph) {
    s = enqueue(st);
    if (s != CS_OK) return s;
  } else {
    if (!same) {
      if (G.exec) cudaGraphExecDestroy(G.exec);
      if (G.graph) cudaGraphDestroy(G.graph);
      G.exec = nullptr; G.graph = nullptr;
      s = ensure_act_maps(ctx, cs_ceil_div(B * (k + 1), 16) * 16);   // host work that must precede capture
      if (s != CS_OK) return s;
      CS_CUDA_OK(ctx, cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeRelaxed));
      s = enqueue(ctx->cap_stream);
      cudaError_t e = cudaStreamEndCapture(ctx->cap_stream, &G.graph);
      if (s == CS_OK && e == cudaSuccess) e = cudaGraphInstantiate(&G.exec, G.graph, 0);
      if (s != CS_OK || e != cudaSuccess) {
        if (G.graph) cudaGraphDestroy(G.graph);
        G.exec = nullptr; G.graph = nullptr;
        if (s != CS_OK) return s;
        CS_CUDA_OK(ctx, e);
      }
      G.hist_dev = hist_dev; G.hist_len_dev = hist_len_dev; G.kv_cache = kv_cache; G.kv_len = kv_len;
      G.B = B; G.stride = stride; G.gamma = gamma; G.k = k; G.policy = (int)policy; G.scripted = script_dev != nullptr;
    }
    CS_CUDA_OK(ctx, cudaGraphLaunch(G.exec, st));
  }
  // ---- device -> host, then step 4 on the host: append what was emitted
  CS_CUDA_OK(ctx, cudaMemcpyAsync(accept_len_host, ctx->loop_accept, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
  CS_CUDA_OK(ctx, cudaMemcpyAsync(out_tokens_host, ctx->loop_out, (size_t)B * (k + 1) * 4, cudaMemcpyDeviceToHost, st));
  CS_CUDA_OK(ctx, cudaStreamSynchronize(st));
  for (int b = 0; b < B; ++b) {
    const int tau = accept_len_host[b];
    if (tau < 0 || tau > k) continue;                  // the device skipped this sequence (status word)
    const int n = hist_len_host[b];
    for (int i = 0; i <= tau; ++i) hist_host[(size_t)b * stride + n + i] = out_tokens_host[(size_t)b * (k + 1) + i];
    hist_len_host[b] = n + tau + 1;
  }
  for (int b = 0; b < B; ++b) G.host_len[b] = hist_len_host[b];
  return CS_OK;
}

void cs_step_host_reset(cs_ctx* ctx) {
  if (ctx != nullptr) ctx->host_step.up_host = nullptr;
}

cs_status cs_debug_drop_tile(cs_ctx* ctx, int k_block) {
  if (ctx == nullptr) return CS_ERR_ARG;
  ctx->debug_drop_kb = k_block < 0 ? -1 : k_block;
  return CS_OK;
}

cs_status cs_kv_truncate(cs_ctx* ctx, int32_t* kv_len, const int32_t* new_len, int B, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (B < 0 || kv_len == nullptr || new_len == nullptr) return fail(ctx, CS_ERR_ARG, "bad argument");
  if (B == 0) return CS_OK;
  cs_launch_truncate(ctx, kv_len, new_len, B, static_cast<cudaStream_t>(stream));
  CS_CUDA_OK(ctx, cudaGetLastError());
  return CS_OK;
}

cs_status cs_prefill(cs_ctx* ctx, const int32_t* hist, const int32_t* hist_len, int B, int stride, int max_len,
                     void* kv_cache, int32_t* kv_len, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (B < 1 || B > ctx->cfg.max_batch || hist == nullptr || hist_len == nullptr || kv_cache == nullptr ||
      kv_len == nullptr || max_len < 0 || stride < max_len)
    return fail(ctx, CS_ERR_ARG, "bad argument");
  if (max_len - 1 > ctx->cfg.max_seq) return fail(ctx, CS_ERR_CAPACITY, "history longer than the KV cache");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int R = CS_MAX_ROWS / B;
  const int total = max_len - 1;   // positions whose K/V are cached
  for (int start = 0; start < total; start += R) {
    const int r = (total - start < R) ? total - start : R;
    ctx->stamp_n = 0;
    cs_launch_prefill_setup(ctx, hist, hist_len, B, stride, start, r, st);
    cs_status s = enqueue_forward(ctx, B, r, kv_cache, false, nullptr, st);
    if (s != CS_OK) { ctx->one_term = false; return s; }
  }
  ctx->one_term = false;
  if (total <= 0) cs_launch_prefill_setup(ctx, hist, hist_len, B, stride, 0, 1, st);   // sets seq_ok
  cs_launch_prefill_finish(ctx, hist_len, kv_len, B, st);
  CS_CUDA_OK(ctx, cudaGetLastError());
  return CS_OK;
}

cs_status cs_loop_begin(cs_ctx* ctx, int32_t* hist, int32_t* hist_len, int B, int stride, void* kv_cache,
                        int32_t* kv_len, int gamma, int k, cs_match_policy policy, int max_new, int eos_id,
                        const int32_t* script, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (B < 1 || B > ctx->cfg.max_batch || k < 0 || k > ctx->cfg.k_max || gamma < 1 || gamma > CS_MAX_GAMMA ||
      max_new < 0 || stride < 1)
    return fail(ctx, CS_ERR_ARG, "B, k, gamma, max_new or stride out of range");
  if (policy != CS_MATCH_LATEST && policy != CS_MATCH_FIRST) return fail(ctx, CS_ERR_ARG, "bad policy");
  if (hist == nullptr || hist_len == nullptr || kv_cache == nullptr || kv_len == nullptr)
    return fail(ctx, CS_ERR_ARG, "NULL argument");
  cs_loop_end(ctx);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  LoopState& L = ctx->loop;
  L.hist = hist; L.hist_len = hist_len; L.B = B; L.stride = stride; L.kv_cache = kv_cache; L.kv_len = kv_len;
  L.gamma = gamma; L.k = k; L.policy = (int)policy; L.max_new = max_new; L.eos_id = eos_id; L.script = script;
  L.use_graph = !ctx->no_graph;
  L.use_index = ctx->match_index != nullptr;
  if (L.use_index) {
    if (ctx->match_index_cap < stride) return fail(ctx, CS_ERR_CAPACITY, "the gamma-gram index is sized for fewer tokens than a history row holds");
    // built afresh from the histories as they stand
    cs_status r = cs_gram_index_reset(ctx->match_index, B, ctx->match_index_cap, st);
    if (r == CS_OK) r = cs_launch_gram_update(ctx->match_index, B, ctx->match_index_cap, hist, hist_len, stride, gamma, 64, ctx->d_status, st);
    if (r != CS_OK) return fail(ctx, r, "index build failed");
  }

  cs_launch_loop_init(ctx, hist_len, kv_len, B, stride, max_new, k, st);
  CS_CUDA_OK(ctx, cudaGetLastError());
  // the activation maps must exist before capture (encoding them is host work)
  cs_status s = ensure_act_maps(ctx, cs_ceil_div(B * (k + 1), 16) * 16);
  if (s != CS_OK) return s;
  if (L.use_graph) {
    // captured on the context's own stream (the legacy default stream cannot capture),
    // replayed on the caller's
    CS_CUDA_OK(ctx, cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeRelaxed));
    s = enqueue_loop_step(ctx, ctx->cap_stream);
    cudaError_t e = cudaStreamEndCapture(ctx->cap_stream, &L.graph);
    if (s != CS_OK) { cs_loop_end(ctx); return s; }
    if (e != cudaSuccess) { cs_loop_end(ctx); CS_CUDA_OK(ctx, e); }
    e = cudaGraphInstantiate(&L.exec, L.graph, 0);
    if (e != cudaSuccess) { cs_loop_end(ctx); CS_CUDA_OK(ctx, e); }
    size_t nodes = 0;
    if (cudaGraphGetNodes(L.graph, nullptr, &nodes) == cudaSuccess) L.graph_nodes = (int)nodes;
    // the same step CS_LOOP_UNROLL times over in one graph, for runs of several steps
    CS_CUDA_OK(ctx, cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeRelaxed));
    for (int i = 0; i < CS_LOOP_UNROLL && s == CS_OK; ++i) s = enqueue_loop_step(ctx, ctx->cap_stream);
    e = cudaStreamEndCapture(ctx->cap_stream, &L.graph_n);
    if (s != CS_OK) { cs_loop_end(ctx); return s; }
    if (e != cudaSuccess) { cs_loop_end(ctx); CS_CUDA_OK(ctx, e); }
    e = cudaGraphInstantiate(&L.exec_n, L.graph_n, 0);
    if (e != cudaSuccess) { cs_loop_end(ctx); CS_CUDA_OK(ctx, e); }
  }
  L.active = true;
  return CS_OK;
}

cs_status cs_loop_steps(cs_ctx* ctx, int n_steps, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (!ctx->loop.active || n_steps < 0) return fail(ctx, CS_ERR_ARG, "no loop in progress");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  for (int i = 0; i < n_steps; ++i) {
    if (ctx->loop.use_graph) {
      if (n_steps - i >= CS_LOOP_UNROLL && ctx->loop.exec_n != nullptr) {
        CS_CUDA_OK(ctx, cudaGraphLaunch(ctx->loop.exec_n, st));
        i += CS_LOOP_UNROLL - 1;
        continue;
      }
      CS_CUDA_OK(ctx, cudaGraphLaunch(ctx->loop.exec, st));
    } else {
      cs_status s = enqueue_loop_step(ctx, st);
      if (s != CS_OK) return s;
    }
  }
  return CS_OK;
}

cs_status cs_loop_poll(cs_ctx* ctx, cs_stats* stats_out, int* n_done_out, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (!ctx->loop.active) return fail(ctx, CS_ERR_ARG, "no loop in progress");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int done = 0;
  CS_CUDA_OK(ctx, cudaMemcpyAsync(&done, ctx->loop_done + ctx->cfg.max_batch, sizeof(int), cudaMemcpyDeviceToHost, st));
  if (stats_out != nullptr)
    CS_CUDA_OK(ctx, cudaMemcpyAsync(stats_out, ctx->loop_stats, sizeof(cs_stats), cudaMemcpyDeviceToHost, st));
  CS_CUDA_OK(ctx, cudaStreamSynchronize(st));
  if (n_done_out != nullptr) *n_done_out = done;
  return cs_sync_status(ctx, stream);
}

cs_status cs_loop_last_step(cs_ctx* ctx, int32_t* match_pos_host, int32_t* draft_len_host, int32_t* accept_len_host,
                            int32_t* out_tokens_host, int32_t* argmax_ids_host, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (!ctx->loop.active) return fail(ctx, CS_ERR_ARG, "no loop in progress");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t B = (size_t)ctx->loop.B, R = (size_t)ctx->loop.k + 1;
  const struct { int32_t* dst; const int* src; size_t n; } copies[5] = {
      {match_pos_host, ctx->loop_mpos, B},        {draft_len_host, ctx->loop_dlen, B},
      {accept_len_host, ctx->loop_accept, B},     {out_tokens_host, ctx->loop_out, B * R},
      {argmax_ids_host, ctx->loop_argmax, B * R}};
  for (const auto& c : copies)
    if (c.dst != nullptr) CS_CUDA_OK(ctx, cudaMemcpyAsync(c.dst, c.src, c.n * 4, cudaMemcpyDeviceToHost, st));
  CS_CUDA_OK(ctx, cudaStreamSynchronize(st));
  return CS_OK;
}

int cs_loop_launches_per_step(const cs_ctx* ctx) {
  return (ctx != nullptr && ctx->loop.active) ? ctx->loop.graph_nodes : 0;
}

void cs_loop_end(cs_ctx* ctx) {
  if (ctx == nullptr) return;
  if (ctx->loop.exec) cudaGraphExecDestroy(ctx->loop.exec);
  if (ctx->loop.graph) cudaGraphDestroy(ctx->loop.graph);
  if (ctx->loop.exec_n) cudaGraphExecDestroy(ctx->loop.exec_n);
  if (ctx->loop.graph_n) cudaGraphDestroy(ctx->loop.graph_n);
  ctx->loop.exec = nullptr;
  ctx->loop.graph = nullptr;
  ctx->loop.exec_n = nullptr;
  ctx->loop.graph_n = nullptr;
  ctx->loop.active = false;
}

cs_status cs_decode_loop(cs_ctx* ctx, int32_t* hist, int32_t* hist_len, int B, int stride, void* kv_cache,
                         int32_t* kv_len, int gamma, int k, cs_match_policy policy, int max_new, int eos_id,
                         const int32_t* script, cs_stats* stats_out, void* stream) {
  cs_status s = cs_loop_begin(ctx, hist, hist_len, B, stride, kv_cache, kv_len, gamma, k, policy, max_new, eos_id,
                              script, stream);
  if (s != CS_OK) return s;
  // every live sequence emits at least one token per step, so max_new steps always suffice
  // A status that concerns single sequences (no room, inconsistent lengths: those sequences
  // were marked finished and left alone) is remembered while the others run on; a CUDA error or
  // a wait that ran out ends the loop.
  const int poll = 4;
  int steps = 0, done = 0;
  cs_status first = CS_OK;
  char first_msg[sizeof(ctx->err)] = "";
  while (true) {
    const int nrun = (max_new - steps < poll) ? max_new - steps : poll;
    if (nrun > 0) s = cs_loop_steps(ctx, nrun, stream);
    steps += nrun;
    if (s != CS_OK) break;
    s = cs_loop_poll(ctx, stats_out, &done, stream);
    if (s == CS_ERR_CAPACITY || s == CS_ERR_ARG) {
      if (first == CS_OK) { first = s; snprintf(first_msg, sizeof(first_msg), "%s", ctx->err); }
      s = CS_OK;
    }
    if (s != CS_OK || done >= B || steps >= max_new) break;
  }
  cs_loop_end(ctx);
  if (s == CS_OK && first != CS_OK) {
    snprintf(ctx->err, sizeof(ctx->err), "%s", first_msg);
    s = first;
  }
  return s;
}

cs_status cs_set_match_index(cs_ctx* ctx, void* index, int capacity_tokens) {
  if (ctx == nullptr || (index != nullptr && capacity_tokens < 1)) return CS_ERR_ARG;
  if (ctx->loop.active) return fail(ctx, CS_ERR_ARG, "the search method cannot change while a loop is in progress");
  ctx->match_index = index;
  ctx->match_index_cap = index != nullptr ? capacity_tokens : 0;
  return CS_OK;
}

cs_status cs_set_stamps(cs_ctx* ctx, unsigned long long* stamps, int capacity) {
  if (ctx == nullptr || capacity < 0) return CS_ERR_ARG;
  if (ctx->loop.active) return fail(ctx, CS_ERR_ARG, "stamps cannot change while a loop is in progress (its graph holds the slots)");
  ctx->stamp_buf = (capacity > 0) ? stamps : nullptr;
  ctx->stamp_cap = (stamps != nullptr) ? capacity : 0;
  ctx->stamp_n = 0;
  // graphs captured earlier hold the old slots
  for (int i = 0; i < CS_VERIFY_GRAPHS; ++i) {
    if (ctx->verify_graphs[i].exec) cudaGraphExecDestroy(ctx->verify_graphs[i].exec);
    if (ctx->verify_graphs[i].graph) cudaGraphDestroy(ctx->verify_graphs[i].graph);
    ctx->verify_graphs[i] = VerifyGraph{};
  }
  if (ctx->host_step.exec) cudaGraphExecDestroy(ctx->host_step.exec);
  if (ctx->host_step.graph) cudaGraphDestroy(ctx->host_step.graph);
  ctx->host_step.exec = nullptr;
  ctx->host_step.graph = nullptr;
  return CS_OK;
}

int cs_stamp_layout(const cs_ctx* ctx, int* family, int capacity) {
  if (ctx == nullptr) return 0;
  for (int i = 0; i < ctx->stamp_n && i < capacity && family != nullptr; ++i) family[i] = ctx->stamp_fam[i];
  return ctx->stamp_n;
}

cs_status cs_linear(cs_ctx* ctx, const void* X, const void* W, int rows, int N, int K, float* Y, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (X == nullptr || W == nullptr || Y == nullptr || rows < 1 || rows > CS_MAX_ROWS || N < 1 || K < 8 || (K % 8))
    return fail(ctx, CS_ERR_ARG, "bad argument");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  GemmPlan g;
  cs_status s = cs_gemm_plan(ctx, &g, W, N, K, true);
  if (s != CS_OK) return s;
  const int n_tok = cs_ceil_div(rows, 16) * 16;
  CUtensorMap tmX;
  if ((s = cs_make_act_map(ctx, &tmX, X, n_tok, K, n_tok)) != CS_OK) return s;
  return cs_launch_gemm(ctx, &g, &tmX, -1, rows, CS_EPI_STORE, Y, nullptr, nullptr, 0, nullptr, nullptr, st);
}

cs_status cs_lm_head(cs_ctx* ctx, const void* X, int rows, int32_t* ids, float* logits_dbg, void* stream) {
  if (ctx == nullptr) return CS_ERR_ARG;
  if (X == nullptr || ids == nullptr || rows < 1 || rows > CS_MAX_ROWS) return fail(ctx, CS_ERR_ARG, "bad argument");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_tok = cs_ceil_div(rows, 16) * 16;
  CUtensorMap tmX;
  cs_status s = cs_make_act_map(ctx, &tmX, X, n_tok, ctx->cfg.d_model, n_tok);
  if (s != CS_OK) return s;
  if ((s = cs_launch_gemm(ctx, &ctx->lm, &tmX, -1, rows, CS_EPI_ARGMAX, logits_dbg, nullptr, nullptr, 0, nullptr, nullptr, st)) != CS_OK) return s;
  cs_launch_tile_reduce(ctx, rows, ids, st);
  CS_CUDA_OK(ctx, cudaGetLastError());
  return CS_OK;
}

}  // extern "C"
