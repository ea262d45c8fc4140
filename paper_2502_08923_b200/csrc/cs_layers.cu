// The small kernels around the GEMMs and the attention of the verification forward
// (Sec. 3.2; App. B.2): block assembly (rows, positions, rotary table), embedding lookup with
// the first RMSNorm, the merge of the attention's key slices, the reduction of the LM-head
// tile maxima with prefix acceptance, KV truncation, and the loop's init and commit steps.
// RoPE, the K/V append, SwiGLU, the residual adds and every later RMSNorm live in the GEMM
// epilogues (cs_gemm.cu); attention is in cs_attn_tc.cu and cs_attn.cu.
#include <math.h>

#include "cs_common.cuh"

namespace {

// ----------------------------------------------------------------- block assembly
// Rows of sequence b: r = 0 is the last accepted token, r = 1..draft_len[b] the draft
// (Sec. 3.2: the speculative tokens are appended to the context).  Rows past the draft
// are dead: they are computed but attend to nothing and write nothing.
__global__ void k_block_setup(const int* __restrict__ last_tok, const int* __restrict__ draft,
                              const int* __restrict__ draft_len, const int* __restrict__ kv_len,
                              const int* __restrict__ skip, int B, int k, int max_seq, int vocab,
                              int half, const double* __restrict__ inv_freq, int* row_tok, int* row_pos,
                              int* row_lim, int* row_write, int* seq_ok, float* rope_cs, int* status,
                              unsigned long long* stamp) {
  CS_PDL_PROLOGUE();
  const int R = k + 1, rows = B * R;
  for (int row = threadIdx.x; row < rows; row += blockDim.x) {
    const int b = row / R, r = row % R;
    int dl = draft_len[b];
    dl = dl < 0 ? 0 : (dl > k ? k : dl);
    const int kv = kv_len[b];
    const bool skipped = (skip != nullptr && skip[b] != 0);
    const bool fits = (kv >= 0 && kv + dl + 1 <= max_seq);
    const bool ok = fits && !skipped;
    if (r == 0) {
      seq_ok[b] = ok ? 1 : 0;
      if (!fits && !skipped) atomicOr(status, CS_DEV_CAPACITY);
    }
    const bool valid = ok && r <= dl;
    int tok = (r == 0 || !valid) ? last_tok[b] : draft[(size_t)b * k + r - 1];
    tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
    row_tok[row] = tok;
    row_pos[row] = (kv < 0 ? 0 : kv) + r;
    row_lim[row] = valid ? kv + r + 1 : 0;
    row_write[row] = valid ? 1 : 0;
  }
  for (int i = threadIdx.x; i < rows * half; i += blockDim.x) {
    const int row = i / half, j = i % half;
    const int b = row / R, r = row % R;
    const int kv = kv_len[b];
    const double ang = (double)((kv < 0 ? 0 : kv) + r) * inv_freq[j];
    double s, c;
    sincos(ang, &s, &c);
    rope_cs[2 * i] = (float)c;
    rope_cs[2 * i + 1] = (float)s;
  }
  if (stamp != nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) cs_stamp_end(stamp);
  }
}

// Forced rows for filling the cache from a history: row r of sequence b is token
// hist[b][start + r]; only positions below hist_len[b] - 1 are computed.
__global__ void k_prefill_setup(const int* __restrict__ hist, const int* __restrict__ hist_len, int B,
                                int stride, int start, int R, int max_seq, int vocab, int half,
                                const double* __restrict__ inv_freq, int* row_tok, int* row_pos,
                                int* row_lim, int* row_write, int* seq_ok, float* rope_cs, int* status) {
  CS_PDL_PROLOGUE();
  const int rows = B * R;
  for (int row = threadIdx.x; row < rows; row += blockDim.x) {
    const int b = row / R, r = row % R;
    const int p = start + r;
    const int n = hist_len[b];
    const bool fits = (n - 1 <= max_seq && n <= stride);
    if (r == 0) {
      seq_ok[b] = fits ? 1 : 0;
      if (!fits) atomicOr(status, CS_DEV_CAPACITY);
    }
    const bool valid = fits && p < n - 1;
    int tok = valid ? hist[(size_t)b * stride + p] : 0;
    tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
    row_tok[row] = tok;
    row_pos[row] = p;
    row_lim[row] = valid ? p + 1 : 0;
    row_write[row] = valid ? 1 : 0;
  }
  for (int i = threadIdx.x; i < rows * half; i += blockDim.x) {
    const int row = i / half, j = i % half;
    const double ang = (double)(start + row % R) * inv_freq[j];
    double s, c;
    sincos(ang, &s, &c);
    rope_cs[2 * i] = (float)c;
    rope_cs[2 * i + 1] = (float)s;
  }
}

// Embedding lookup and the first RMSNorm in one pass: x = E[token] (fp32 residual stream) and
// xn = x * rsqrt(mean(x^2) + eps) * g as two bf16 terms (hi, lo).  One CTA per row; the row is
// read once and kept in registers (up to 4 float4 per thread).  Every later norm is folded
// into the GEMMs around it.
constexpr int kNormThreads = 1024;
__global__ void __launch_bounds__(kNormThreads)
k_embed_rmsnorm(const __nv_bfloat16* __restrict__ E, const int* __restrict__ row_tok, float* __restrict__ x, int d,
                const __nv_bfloat16* __restrict__ gain, float eps, __nv_bfloat16* __restrict__ xn,
                __nv_bfloat16* __restrict__ xn_lo, unsigned long long* stamp) {
  CS_PDL_PROLOGUE();
  const int row = blockIdx.x;
  const __nv_bfloat16* er = E + (size_t)row_tok[row] * d;
  float* xr = x + (size_t)row * d;
  auto fetch = [&](int i) {
    const uint2 w = *reinterpret_cast<const uint2*>(er + i);          // four bf16
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w.y));
    const float4 v = make_float4(a.x, a.y, b.x, b.y);
    *reinterpret_cast<float4*>(xr + i) = v;
    return v;
  };
  float4 v[4];
  float ss = 0.f;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int i = (q * kNormThreads + threadIdx.x) * 4;
    v[q] = (i < d) ? fetch(i) : make_float4(0.f, 0.f, 0.f, 0.f);
    ss += v[q].x * v[q].x + v[q].y * v[q].y + v[q].z * v[q].z + v[q].w * v[q].w;
  }
  for (int i = 4 * kNormThreads * 4 + threadIdx.x * 4; i < d; i += kNormThreads * 4) {   // d > 16384
    const float4 w = fetch(i);
    ss += w.x * w.x + w.y * w.y + w.z * w.z + w.w * w.w;
  }
  __shared__ float red[32];
  __shared__ float s_scale;
  for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x < 32) {
    float t = red[threadIdx.x];
    for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
    if (threadIdx.x == 0) s_scale = rsqrtf(t / (float)d + eps);
  }
  __syncthreads();
  const float sc = s_scale;
  auto emit = [&](int i, const float4& w) {
    const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(gain + i));
    const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(gain + i + 2));
    const float y0 = w.x * sc * g0.x, y1 = w.y * sc * g0.y, y2 = w.z * sc * g1.x, y3 = w.w * sc * g1.y;
    const __nv_bfloat162 o0 = __floats2bfloat162_rn(y0, y1), o1 = __floats2bfloat162_rn(y2, y3);
    *reinterpret_cast<__nv_bfloat162*>(xn + (size_t)row * d + i) = o0;
    *reinterpret_cast<__nv_bfloat162*>(xn + (size_t)row * d + i + 2) = o1;
    // second term: what the first rounding lost
    const float2 h0 = __bfloat1622float2(o0), h1 = __bfloat1622float2(o1);
    *reinterpret_cast<__nv_bfloat162*>(xn_lo + (size_t)row * d + i) = __floats2bfloat162_rn(y0 - h0.x, y1 - h0.y);
    *reinterpret_cast<__nv_bfloat162*>(xn_lo + (size_t)row * d + i + 2) = __floats2bfloat162_rn(y2 - h1.x, y3 - h1.y);
  };
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int i = (q * kNormThreads + threadIdx.x) * 4;
    if (i < d) emit(i, v[q]);
  }
  for (int i = 4 * kNormThreads * 4 + threadIdx.x * 4; i < d; i += kNormThreads * 4)
    emit(i, *reinterpret_cast<const float4*>(xr + i));
  if (stamp != nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) cs_stamp_end(stamp);
  }
}

// Combine the key slices: o = sum_s o_s e^(m_s - M) / sum_s l_s e^(m_s - M).  NS = an upper
// bound of the slice count known at compile time, so the loads and the sum are unrolled to it.
template <int NS>
__global__ void k_attn_merge(const float* __restrict__ in_o, const float* __restrict__ in_ml, int nsplit,
                             int rows, int H, int Dh, __nv_bfloat16* __restrict__ attn_out,
                             unsigned long long* stamp) {
  CS_PDL_PROLOGUE();
  const int row = blockIdx.x, h = blockIdx.y, dd = threadIdx.x;
  const int lane = threadIdx.x & 31;
  // all partial outputs of this (row, head, dim) are requested at once, so their latencies
  // overlap each other and the weight computation below
  float v[NS];
  {
    const size_t stride = (size_t)rows * H * Dh;
    const float* src = in_o + ((size_t)row * H + h) * Dh + dd;
#pragma unroll
    for (int s = 0; s < NS; ++s) v[s] = (s < nsplit) ? src[(size_t)s * stride] : 0.f;
  }
  // every warp works out the slice weights e^(m_s - M) / L itself: lane s owns slices s, s+32
  float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;
  if (lane < nsplit) {
    const size_t base = ((size_t)lane * rows + row) * H + h;
    m0 = in_ml[base * 2]; l0 = in_ml[base * 2 + 1];
  }
  if (NS > 32 && lane + 32 < nsplit) {
    const size_t base = ((size_t)(lane + 32) * rows + row) * H + h;
    m1 = in_ml[base * 2]; l1 = in_ml[base * 2 + 1];
  }
  float M = fmaxf(m0, m1);
  for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
  float w0 = (m0 == -INFINITY) ? 0.f : expf(m0 - M), w1 = (m1 == -INFINITY) ? 0.f : expf(m1 - M);
  float L = l0 * w0 + l1 * w1;
  for (int off = 16; off > 0; off >>= 1) L += __shfl_xor_sync(0xffffffffu, L, off);
  const float inv = L > 0.f ? 1.f / L : 0.f;
  w0 *= inv; w1 *= inv;
  float acc = 0.f;
#pragma unroll
  for (int s = 0; s < NS; ++s) {
    const float w = __shfl_sync(0xffffffffu, s < 32 ? w0 : w1, s & 31);
    acc = fmaf(v[s], w, acc);
  }
  const __nv_bfloat16 hi = __float2bfloat16_rn(acc);
  attn_out[((size_t)row * H + h) * Dh + dd] = hi;
  attn_out[((size_t)(CS_MAX_ROWS + row) * H + h) * Dh + dd] = __float2bfloat16_rn(acc - __bfloat162float(hi));
  if (stamp != nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) cs_stamp_end(stamp);
  }
}

// ------------------------------------------------------------------ acceptance
// Reduce the LM-head tile maxima to the greedy token of each row (lowest id on ties),
// then accept the longest prefix of the draft that agrees with the target tokens and
// emit it plus one extra token (Sec. 3.2; App. B.2).  One CTA per sequence.
__global__ void __launch_bounds__(512)
k_accept(const float* __restrict__ tile_max, const int* __restrict__ tile_idx, int tiles, int tile_stride,
         int k, const int* __restrict__ draft, const int* __restrict__ draft_len,
         const int* __restrict__ seq_ok, const int* __restrict__ script, int script_stride,
         const int* __restrict__ script_off, int script_limit, int* __restrict__ accept_len,
         int* __restrict__ out_tokens, int* __restrict__ argmax_ids, int* __restrict__ kv_len,
         int update_kv, unsigned long long* stamp) {
  CS_PDL_PROLOGUE();
  const int b = blockIdx.x, R = k + 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  __shared__ int s_arg[CS_MAX_ROWS];
  int dl = draft_len[b];
  dl = dl < 0 ? 0 : (dl > k ? k : dl);
  const bool ok = seq_ok[b] != 0;
  // Greedy token of every live row: one warp per row, its lanes striding over the tile maxima (all
  // of a lane's loads are independent, so their latencies overlap), then a shuffle reduction.
  for (int r = warp; r < R; r += nwarps) {
    float val = -INFINITY;
    int idx = INT32_MAX;
    if (ok && r <= dl) {
      const int row = b * R + r;
      for (int t = lane; t < tiles; t += 32) {
        const float v = tile_max[(size_t)row * tile_stride + t];
        const int id = tile_idx[(size_t)row * tile_stride + t];
        if (v > val || (v == val && id < idx)) { val = v; idx = id; }
      }
      for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, val, off);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, off);
        if (ov > val || (ov == val && oi < idx)) { val = ov; idx = oi; }
      }
    }
    if (lane == 0) s_arg[r] = (ok && r <= dl && idx != INT32_MAX) ? idx : -1;
  }
  __syncthreads();
  for (int r = threadIdx.x; r < R; r += blockDim.x) argmax_ids[(size_t)b * R + r] = s_arg[r];
  if (threadIdx.x == 0) {
    if (!ok) {
      accept_len[b] = -1;
      for (int r = 0; r < R; ++r) out_tokens[(size_t)b * R + r] = -1;
      cs_stamp_end(stamp);
      return;
    }
    const int off = (script != nullptr && script_off != nullptr) ? script_off[b] : 0;
    int tau = 0;
    bool open = true;
    for (int r = 0; r < R; ++r) {
      int tgt = s_arg[r];
      if (script != nullptr) tgt = (off + r < script_limit) ? script[(size_t)b * script_stride + off + r] : -1;
      if (r > dl) tgt = -1;
      // row r's target is emitted iff all earlier draft tokens were accepted
      out_tokens[(size_t)b * R + r] = open ? tgt : -1;
      if (open) {
        if (r < dl && draft[(size_t)b * k + r] == tgt) tau = r + 1; else open = false;
      }
    }
    accept_len[b] = tau;
    if (update_kv) kv_len[b] += tau + 1;
    cs_stamp_end(stamp);
  }
}

// Greedy token of each row from the LM head's per-tile (max, id) pairs (lowest id on ties).
__global__ void __launch_bounds__(128)
k_tile_reduce(const float* __restrict__ tile_max, const int* __restrict__ tile_idx, int tiles, int tile_stride,
              int* __restrict__ ids) {
  CS_PDL_PROLOGUE();
  const int row = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float val = -INFINITY;
  int idx = INT32_MAX;
  for (int t = threadIdx.x; t < tiles; t += 128) {
    const float v = tile_max[(size_t)row * tile_stride + t];
    const int id = tile_idx[(size_t)row * tile_stride + t];
    if (v > val || (v == val && id < idx)) { val = v; idx = id; }
  }
  __shared__ float sv[4];
  __shared__ int si[4];
  for (int off = 16; off > 0; off >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, val, off);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, off);
    if (ov > val || (ov == val && oi < idx)) { val = ov; idx = oi; }
  }
  if (lane == 0) { sv[warp] = val; si[warp] = idx; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 4; ++w)
      if (sv[w] > val || (sv[w] == val && si[w] < idx)) { val = sv[w]; idx = si[w]; }
    ids[row] = (idx == INT32_MAX) ? -1 : idx;
  }
}

__global__ void k_truncate(int* kv_len, const int* new_len, int B, int* status) {
  CS_PDL_PROLOGUE();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int nl = new_len[b];
  if (nl < 0 || nl > kv_len[b]) atomicOr(status, CS_DEV_BADARG);
  else kv_len[b] = nl;
}

__global__ void k_prefill_finish(const int* hist_len, const int* seq_ok, int* kv_len, int B) {
  CS_PDL_PROLOGUE();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B && seq_ok[b]) kv_len[b] = max(0, hist_len[b] - 1);
}

// ------------------------------------------------------------------ loop bookkeeping
__global__ void k_loop_init(const int* hist_len, const int* kv_len, int B, int stride, int max_new, int k,
                            int max_seq, int max_batch, int* emitted, int* done,
                            unsigned long long* stats, int* status) {
  CS_PDL_PROLOGUE();
  const int t = threadIdx.x;
  for (int i = t; i < (int)(sizeof(cs_stats) / 8); i += blockDim.x) stats[i] = 0ull;
  __shared__ int s_done;
  if (t == 0) s_done = 0;
  __syncthreads();
  for (int b = t; b < B; b += blockDim.x) {
    const int n = hist_len[b];
    const bool fits = n >= 1 && n + max_new <= stride && n + max_new + k <= max_seq;
    const bool consistent = kv_len[b] == n - 1;
    emitted[b] = 0;
    int d = 0;
    if (!fits) { atomicOr(status, CS_DEV_CAPACITY); d = 1; }
    else if (!consistent) { atomicOr(status, CS_DEV_BADARG); d = 1; }
    else if (max_new <= 0) d = 1;
    done[b] = d;
    if (d) atomicAdd(&s_done, 1);
  }
  __syncthreads();
  if (t == 0) done[max_batch] = s_done;
}

// Append the step's tokens to the history (App. B.3 step 4), clip at max_new, stop at
// EOS in real mode, advance the lengths (the KV truncation of App. B.2) and count.
__global__ void k_loop_commit(int* hist, int* hist_len, int B, int stride, int* kv_len, int k, int max_new,
                              int eos_id, int scripted, const int* accept, const int* out, const int* mpos,
                              int* emitted, int* done, int max_batch, unsigned long long* stats,
                              unsigned long long* stamp) {
  CS_PDL_PROLOGUE();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b == 0) cs_stamp_end(stamp);   // (the kernel is a few dozen instructions: its start stands for its end)
  if (b >= B || done[b]) return;
  cs_stats* st = reinterpret_cast<cs_stats*>(stats);
  const int tau = accept[b];
  if (tau < 0) {            // the step skipped this sequence (capacity): it stops here
    done[b] = 1;
    atomicAdd(&done[max_batch], 1);
    return;
  }
  const int R = k + 1;
  const int n = hist_len[b], e = emitted[b];
  int c = min(tau + 1, max_new - e);
  bool fin = false;
  if (!scripted && eos_id >= 0) {
    for (int i = 0; i < c; ++i)
      if (out[(size_t)b * R + i] == eos_id) { c = i + 1; fin = true; break; }
  }
  for (int i = 0; i < c; ++i) hist[(size_t)b * stride + n + i] = out[(size_t)b * R + i];
  hist_len[b] = n + c;
  kv_len[b] = n + c - 1;
  emitted[b] = e + c;
  if (e + c >= max_new) fin = true;
  atomicAdd((unsigned long long*)&st->steps, 1ull);
  atomicAdd((unsigned long long*)&st->emitted, (unsigned long long)c);
  if (mpos[b] >= 0) {
    atomicAdd((unsigned long long*)&st->attempts, 1ull);
    atomicAdd((unsigned long long*)&st->accepted, (unsigned long long)(c - 1));
    atomicAdd((unsigned long long*)&st->tau_hist[min(c - 1, CS_TAU_HIST - 1)], 1ull);
  } else {
    atomicAdd((unsigned long long*)&st->no_match, 1ull);
  }
  if (fin) {
    done[b] = 1;
    atomicAdd(&done[max_batch], 1);
  }
}

}  // namespace

void cs_launch_block_setup(cs_ctx* ctx, const int32_t* last_tok, const int32_t* draft,
                           const int32_t* draft_len, const int32_t* kv_len, const int32_t* skip, int B,
                           int k, cudaStream_t st) {
  const cs_model_config& c = ctx->cfg;
  cs_launch_pdl(k_block_setup, dim3(1), dim3(256), 0, st, last_tok, draft, draft_len, kv_len, skip, B, k, c.max_seq,
                c.vocab, c.head_dim / 2, ctx->inv_freq, ctx->row_tok, ctx->row_pos, ctx->row_lim, ctx->row_write,
                ctx->seq_ok, ctx->rope_cs, ctx->d_status, cs_next_stamp(ctx, CS_FAM_OTHER));
}

void cs_launch_prefill_setup(cs_ctx* ctx, const int32_t* hist, const int32_t* hist_len, int B, int stride,
                             int start, int R, cudaStream_t st) {
  const cs_model_config& c = ctx->cfg;
  cs_launch_pdl(k_prefill_setup, dim3(1), dim3(256), 0, st, hist, hist_len, B, stride, start, R, c.max_seq, c.vocab,
                c.head_dim / 2, ctx->inv_freq, ctx->row_tok, ctx->row_pos, ctx->row_lim, ctx->row_write, ctx->seq_ok,
                ctx->rope_cs, ctx->d_status);
}

void cs_launch_embed_rmsnorm(cs_ctx* ctx, const __nv_bfloat16* gain, int rows, cudaStream_t st) {
  cs_launch_pdl(k_embed_rmsnorm, dim3(rows), dim3(kNormThreads), 0, st, ctx->embed, ctx->row_tok, ctx->x, ctx->cfg.d_model, gain,
                ctx->cfg.rms_eps, ctx->xn, ctx->xn + (size_t)CS_MAX_ROWS * ctx->cfg.d_model,
                cs_next_stamp(ctx, CS_FAM_OTHER));
}

void cs_launch_attn_merge(cs_ctx* ctx, int nsplit, int rows, cudaStream_t st) {
  const cs_model_config& c = ctx->cfg;
  auto kernel = nsplit <= 1 ? k_attn_merge<1> : nsplit <= 2 ? k_attn_merge<2> : nsplit <= 4 ? k_attn_merge<4>
              : nsplit <= 8 ? k_attn_merge<8> : nsplit <= 16 ? k_attn_merge<16> : nsplit <= 32 ? k_attn_merge<32>
              : nsplit <= 48 ? k_attn_merge<48> : k_attn_merge<64>;
  cs_launch_pdl(kernel, dim3(rows, c.n_heads), dim3(c.head_dim), 0, st, ctx->attn_o, ctx->attn_ml, nsplit, rows,
                c.n_heads, c.head_dim, ctx->attn_out, cs_next_stamp(ctx, CS_FAM_MERGE));
}

void cs_launch_accept(cs_ctx* ctx, int B, int k, const int32_t* draft, const int32_t* draft_len,
                      const int32_t* script, int script_stride, const int32_t* script_off, int script_limit,
                      int32_t* accept_len, int32_t* out_tokens, int32_t* argmax_ids, int32_t* kv_len,
                      int update_kv, cudaStream_t st) {
  cs_launch_pdl(k_accept, dim3(B), dim3(512), 0, st, ctx->tile_max, ctx->tile_idx,
                cs_ceil_div(ctx->cfg.vocab, CS_GEMM_BM), cs_ceil_div(ctx->cfg.vocab, CS_GEMM_BM), k, draft, draft_len, ctx->seq_ok, script,
                script_stride, script_off, script_limit, accept_len, out_tokens, argmax_ids, kv_len, update_kv,
                cs_next_stamp(ctx, CS_FAM_OTHER));
}

void cs_launch_tile_reduce(cs_ctx* ctx, int rows, int32_t* ids, cudaStream_t st) {
  cs_launch_pdl(k_tile_reduce, dim3(rows), dim3(128), 0, st, ctx->tile_max, ctx->tile_idx,
                cs_ceil_div(ctx->cfg.vocab, CS_GEMM_BM), cs_ceil_div(ctx->cfg.vocab, CS_GEMM_BM), ids);
}

void cs_launch_truncate(cs_ctx* ctx, int32_t* kv_len, const int32_t* new_len, int B, cudaStream_t st) {
  cs_launch_pdl(k_truncate, dim3(cs_ceil_div(B, 128)), dim3(128), 0, st, kv_len, new_len, B, ctx->d_status);
}

void cs_launch_prefill_finish(cs_ctx* ctx, const int32_t* hist_len, int32_t* kv_len, int B, cudaStream_t st) {
  cs_launch_pdl(k_prefill_finish, dim3(cs_ceil_div(B, 128)), dim3(128), 0, st, hist_len, ctx->seq_ok, kv_len, B);
}

void cs_launch_loop_init(cs_ctx* ctx, const int32_t* hist_len, const int32_t* kv_len, int B, int stride,
                         int max_new, int k, cudaStream_t st) {
  cs_launch_pdl(k_loop_init, dim3(1), dim3(256), 0, st, hist_len, kv_len, B, stride, max_new, k, ctx->cfg.max_seq,
                ctx->cfg.max_batch, ctx->loop_emitted, ctx->loop_done, ctx->loop_stats, ctx->d_status);
}

void cs_launch_loop_commit(cs_ctx* ctx, int32_t* hist, int32_t* hist_len, int B, int stride, int32_t* kv_len,
                           int k, int max_new, int eos_id, int scripted, cudaStream_t st) {
  cs_launch_pdl(k_loop_commit, dim3(cs_ceil_div(B, 128)), dim3(128), 0, st, hist, hist_len, B, stride, kv_len, k,
                max_new, eos_id, scripted, ctx->loop_accept, ctx->loop_out, ctx->loop_mpos, ctx->loop_emitted,
                ctx->loop_done, ctx->cfg.max_batch, ctx->loop_stats, cs_next_stamp(ctx, CS_FAM_OTHER));
}
