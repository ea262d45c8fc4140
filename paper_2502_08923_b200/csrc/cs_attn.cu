// Causal block attention of the verification forward over the bf16 KV cache (Sec. 3.2;
// App. B.2): the (k+1) block rows of the G query heads that share one KV head form a small
// query tile (44 rows for k = 10, G = 4) that is multiplied against a slice of the cached
// keys/values.
//
// One CTA = one (sequence, KV head), one slice of the key range (split-KV) and up to 64
// query rows; each of its four warps owns 16 query rows and runs a register-resident
// flash-attention loop on bf16 tensor-core MMAs (m16n8k16, fp32 accumulation): S = Q K^T,
// running row max / sum, O += P V; Q and P enter the MMAs as two bf16 terms each (value =
// hi + lo), so only K and V - which the cache stores in bf16 - are rounded.  K and V tiles of 64 keys stream
// through a double-buffered cp.async pipeline in shared memory (rows padded by 16 bytes so
// that fragment loads and ldmatrix are bank-conflict free).  Each slice writes its
// un-normalised output and (max, sum); k_attn_merge combines the slices.
#include <stdlib.h>

#include "cs_common.cuh"

namespace {

constexpr int kThreads = 128;
constexpr int kKeys = 64;      // keys per tile
constexpr int kStages = 2;
constexpr int kRowsPerCta = 64;

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, int src_bytes) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(s));
}
// (lo, hi) as a leading bf16 pair plus the bf16 pair of what that rounding lost
__device__ __forceinline__ void pack_two(float lo, float hi, uint32_t& first, uint32_t& second) {
  const __nv_bfloat162 a = __floats2bfloat162_rn(lo, hi);
  const float2 af = __bfloat1622float2(a);
  const __nv_bfloat162 b = __floats2bfloat162_rn(lo - af.x, hi - af.y);
  first = *reinterpret_cast<const uint32_t*>(&a);
  second = *reinterpret_cast<const uint32_t*>(&b);
}

template <int DH>
__global__ void __launch_bounds__(kThreads)
k_attn_mma(const __nv_bfloat16* __restrict__ qbuf, const __nv_bfloat16* __restrict__ kv,
           const int* __restrict__ row_lim, int layer, int R, int H, int Hkv, int max_batch, int max_seq,
           int nsplit, float scale_log2e, float* __restrict__ out_o, float* __restrict__ out_ml, int rows,
           unsigned long long* stamp) {
  CS_PDL_PROLOGUE();
  constexpr int STRIDE = DH + 8;          // bf16 elements per shared-memory row
  constexpr int KSTEPS = DH / 16;         // MMA k-steps of the QK^T product
  constexpr int NB_S = kKeys / 8;         // 8-key column blocks of S
  constexpr int NB_O = DH / 8;            // 8-dim column blocks of O
  constexpr int CPR = DH / 8;             // 16-byte chunks per K/V row
  extern __shared__ __align__(16) uint8_t smem_raw[];
  __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem_raw);            // [stages][keys][STRIDE]
  __nv_bfloat16* Vs = Ks + kStages * kKeys * STRIDE;
  __shared__ int s_lmax;

  const int G = H / Hkv;
  const int b = blockIdx.x / Hkv, kvh = blockIdx.x % Hkv;
  const int split = blockIdx.y, rg = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int nq = G * R;

  // longest key range any row of this sequence's block attends to
  if (threadIdx.x == 0) s_lmax = 0;
  __syncthreads();
  {
    int lm = 0;
    for (int r = threadIdx.x; r < R; r += kThreads) lm = max(lm, row_lim[b * R + r]);
    lm = __reduce_max_sync(0xffffffffu, lm);
    if (lane == 0 && lm > 0) atomicMax(&s_lmax, lm);
  }
  __syncthreads();
  const int lmax = s_lmax;
  const int ntiles = (lmax + kKeys - 1) / kKeys;
  const int tps = (ntiles + nsplit - 1) / nsplit;
  const int t0 = split * tps, t1 = min(ntiles, t0 + tps);

  // the two query rows this thread holds fragments of
  const int q_lo = rg * kRowsPerCta + warp * 16 + g, q_hi = q_lo + 8;
  const bool v_lo = q_lo < nq, v_hi = q_hi < nq;
  const int grow_lo = v_lo ? b * R + q_lo % R : 0, grow_hi = v_hi ? b * R + q_hi % R : 0;
  const int head_lo = v_lo ? kvh * G + q_lo / R : 0, head_hi = v_hi ? kvh * G + q_hi / R : 0;
  const int lim_lo = v_lo ? row_lim[grow_lo] : 0, lim_hi = v_hi ? row_lim[grow_hi] : 0;

  const __nv_bfloat16* Kg = kv + ((((size_t)layer * 2 + 0) * max_batch + b) * Hkv + kvh) * (size_t)max_seq * DH;
  const __nv_bfloat16* Vg = kv + ((((size_t)layer * 2 + 1) * max_batch + b) * Hkv + kvh) * (size_t)max_seq * DH;

  auto load_tile = [&](int tile, int stage) {
    const int key0 = tile * kKeys;
    __nv_bfloat16* kd = Ks + stage * kKeys * STRIDE;
    __nv_bfloat16* vd = Vs + stage * kKeys * STRIDE;
    for (int c = threadIdx.x; c < kKeys * CPR; c += kThreads) {
      const int j = c / CPR, cc = c % CPR;
      const int key = key0 + j;
      const int nbytes = key < lmax ? 16 : 0;             // keys past the longest row are zero-filled
      const size_t src = (size_t)min(key, max_seq - 1) * DH + cc * 8;
      cp_async16(kd + j * STRIDE + cc * 8, Kg + src, nbytes);
      cp_async16(vd + j * STRIDE + cc * 8, Vg + src, nbytes);
    }
  };

  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  float o[NB_O][4];
#pragma unroll
  for (int nd = 0; nd < NB_O; ++nd) { o[nd][0] = 0.f; o[nd][1] = 0.f; o[nd][2] = 0.f; o[nd][3] = 0.f; }

  if (t0 < t1) load_tile(t0, 0);
  cp_async_commit();
  // (the first K/V tile is already on its way while the query fragments are fetched)
  // queries come as two bf16 terms (q = qa + qb): two MMAs give the product of the fp32 query
  uint32_t qa[KSTEPS][4], qb[KSTEPS][4];
  {
    const __nv_bfloat16* ql = qbuf + ((size_t)grow_lo * H + head_lo) * DH;
    const __nv_bfloat16* qh = qbuf + ((size_t)grow_hi * H + head_hi) * DH;
    const size_t second = (size_t)CS_MAX_ROWS * H * DH;
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
      qa[ks][0] = v_lo ? *reinterpret_cast<const uint32_t*>(ql + ks * 16 + 2 * t) : 0u;
      qa[ks][1] = v_hi ? *reinterpret_cast<const uint32_t*>(qh + ks * 16 + 2 * t) : 0u;
      qa[ks][2] = v_lo ? *reinterpret_cast<const uint32_t*>(ql + ks * 16 + 8 + 2 * t) : 0u;
      qa[ks][3] = v_hi ? *reinterpret_cast<const uint32_t*>(qh + ks * 16 + 8 + 2 * t) : 0u;
      qb[ks][0] = v_lo ? *reinterpret_cast<const uint32_t*>(ql + second + ks * 16 + 2 * t) : 0u;
      qb[ks][1] = v_hi ? *reinterpret_cast<const uint32_t*>(qh + second + ks * 16 + 2 * t) : 0u;
      qb[ks][2] = v_lo ? *reinterpret_cast<const uint32_t*>(ql + second + ks * 16 + 8 + 2 * t) : 0u;
      qb[ks][3] = v_hi ? *reinterpret_cast<const uint32_t*>(qh + second + ks * 16 + 8 + 2 * t) : 0u;
    }
  }

  for (int tile = t0; tile < t1; ++tile) {
    const int stage = (tile - t0) & 1;
    if (tile + 1 < t1) load_tile(tile + 1, stage ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    const __nv_bfloat16* kt = Ks + stage * kKeys * STRIDE;
    const __nv_bfloat16* vt = Vs + stage * kKeys * STRIDE;
    const int key0 = tile * kKeys;

    // S = Q K^T for this warp's 16 rows and the tile's 64 keys
    float s[NB_S][4];
#pragma unroll
    for (int nb = 0; nb < NB_S; ++nb) {
      s[nb][0] = 0.f; s[nb][1] = 0.f; s[nb][2] = 0.f; s[nb][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        const __nv_bfloat16* kp = kt + (nb * 8 + g) * STRIDE + ks * 16 + 2 * t;
        const uint32_t k0 = *reinterpret_cast<const uint32_t*>(kp), k1 = *reinterpret_cast<const uint32_t*>(kp + 8);
        mma_bf16(s[nb], qa[ks], k0, k1);
        mma_bf16(s[nb], qb[ks], k0, k1);
      }
    }
    // scale (log2 domain), causal mask, running max
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
    for (int nb = 0; nb < NB_S; ++nb) {
      const int key = key0 + nb * 8 + 2 * t;
      s[nb][0] = (key < lim_lo) ? s[nb][0] * scale_log2e : -INFINITY;
      s[nb][1] = (key + 1 < lim_lo) ? s[nb][1] * scale_log2e : -INFINITY;
      s[nb][2] = (key < lim_hi) ? s[nb][2] * scale_log2e : -INFINITY;
      s[nb][3] = (key + 1 < lim_hi) ? s[nb][3] * scale_log2e : -INFINITY;
      mx_lo = fmaxf(mx_lo, fmaxf(s[nb][0], s[nb][1]));
      mx_hi = fmaxf(mx_hi, fmaxf(s[nb][2], s[nb][3]));
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float c_lo = (m_lo == -INFINITY) ? 0.f : exp2f(m_lo - mn_lo);
    const float c_hi = (m_hi == -INFINITY) ? 0.f : exp2f(m_hi - mn_hi);
    m_lo = mn_lo; m_hi = mn_hi;
    float ps_lo = 0.f, ps_hi = 0.f;
#pragma unroll
    for (int nb = 0; nb < NB_S; ++nb) {
      s[nb][0] = (s[nb][0] == -INFINITY) ? 0.f : exp2f(s[nb][0] - mn_lo);
      s[nb][1] = (s[nb][1] == -INFINITY) ? 0.f : exp2f(s[nb][1] - mn_lo);
      s[nb][2] = (s[nb][2] == -INFINITY) ? 0.f : exp2f(s[nb][2] - mn_hi);
      s[nb][3] = (s[nb][3] == -INFINITY) ? 0.f : exp2f(s[nb][3] - mn_hi);
      ps_lo += s[nb][0] + s[nb][1];
      ps_hi += s[nb][2] + s[nb][3];
    }
    l_lo = l_lo * c_lo + ps_lo;     // per-thread share of the row sum; the quad is summed at the end
    l_hi = l_hi * c_hi + ps_hi;
#pragma unroll
    for (int nd = 0; nd < NB_O; ++nd) { o[nd][0] *= c_lo; o[nd][1] *= c_lo; o[nd][2] *= c_hi; o[nd][3] *= c_hi; }

    // O += P V: the S accumulators are already laid out as the A fragments of the next MMA
#pragma unroll
    for (int j = 0; j < kKeys / 16; ++j) {
      // softmax weights as two bf16 terms as well
      uint32_t pa[4], pb[4];
      pack_two(s[2 * j][0], s[2 * j][1], pa[0], pb[0]);
      pack_two(s[2 * j][2], s[2 * j][3], pa[1], pb[1]);
      pack_two(s[2 * j + 1][0], s[2 * j + 1][1], pa[2], pb[2]);
      pack_two(s[2 * j + 1][2], s[2 * j + 1][3], pa[3], pb[3]);
#pragma unroll
      for (int nd = 0; nd < NB_O; nd += 2) {
        // four transposed 8x8 blocks of V: keys 16j..16j+15, dims nd*8 .. nd*8+15
        uint32_t vb[4];
        const int mi = lane >> 3, r8 = lane & 7;
        ldmatrix_x4_trans(vb, vt + (j * 16 + (mi & 1) * 8 + r8) * STRIDE + (nd + (mi >> 1)) * 8);
        mma_bf16(o[nd], pa, vb[0], vb[1]);
        mma_bf16(o[nd], pb, vb[0], vb[1]);
        mma_bf16(o[nd + 1], pa, vb[2], vb[3]);
        mma_bf16(o[nd + 1], pb, vb[2], vb[3]);
      }
    }
    __syncthreads();   // everyone is done with this stage before it is refilled
  }
  cp_async_wait<0>();

  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
  // un-normalised partial result of this key slice; (max, sum) in the natural-log domain
  constexpr float kLn2 = 0.6931471805599453f;
  if (v_lo) {
    const size_t base = ((size_t)split * rows + grow_lo) * H + head_lo;
#pragma unroll
    for (int nd = 0; nd < NB_O; ++nd)
      *reinterpret_cast<float2*>(out_o + base * DH + nd * 8 + 2 * t) = make_float2(o[nd][0], o[nd][1]);
    if (t == 0) { out_ml[base * 2] = m_lo * kLn2; out_ml[base * 2 + 1] = l_lo; }
  }
  if (v_hi) {
    const size_t base = ((size_t)split * rows + grow_hi) * H + head_hi;
#pragma unroll
    for (int nd = 0; nd < NB_O; ++nd)
      *reinterpret_cast<float2*>(out_o + base * DH + nd * 8 + 2 * t) = make_float2(o[nd][2], o[nd][3]);
    if (t == 0) { out_ml[base * 2] = m_hi * kLn2; out_ml[base * 2 + 1] = l_hi; }
  }
  if (stamp != nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) cs_stamp_end(stamp);
  }
}

template <int DH>
int launch(cs_ctx* ctx, const void* kv_cache, int layer, int B, int R, cudaStream_t st) {
  const cs_model_config& c = ctx->cfg;
  const int G = c.n_heads / c.n_kv_heads;
  const int rgs = cs_ceil_div(G * R, kRowsPerCta);
  // enough key slices to give every SM about two CTAs, never more than the workspace holds
  int nsplit = cs_ceil_div(2 * ctx->num_sms, B * c.n_kv_heads * rgs);
  if (nsplit > ctx->attn_splits) nsplit = ctx->attn_splits;
  if (nsplit < 1) nsplit = 1;
  const size_t smem = (size_t)2 * kStages * kKeys * (DH + 8) * 2;
  if (!(ctx->attn_mma_attr_set & (1u << (DH / 32)))) {
    cudaFuncSetAttribute(k_attn_mma<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    ctx->attn_mma_attr_set |= 1u << (DH / 32);
  }
  const float scale_log2e = 1.4426950408889634f / sqrtf((float)DH);
  cs_launch_pdl(k_attn_mma<DH>, dim3(B * c.n_kv_heads, nsplit, rgs), dim3(kThreads), smem, st, ctx->qbuf,
                static_cast<const __nv_bfloat16*>(kv_cache), ctx->row_lim, layer, R, c.n_heads, c.n_kv_heads,
                c.max_batch, c.max_seq, nsplit, scale_log2e, ctx->attn_o, ctx->attn_ml, B * R,
                cs_next_stamp(ctx, CS_FAM_ATTENTION));
  return nsplit;
}

}  // namespace

int cs_attention_tc_group_rows(const cs_ctx* ctx, int R);   // cs_attn_tc.cu

void cs_launch_attention(cs_ctx* ctx, const void* kv_cache, int layer, int B, int R, cudaStream_t st) {
  // head_dim 128 runs on the tcgen05 kernels: the one with the query rows as M while a CTA walks
  // at most two key tiles (a 4k context at batch 1: a latency chain, one tile on each of two CTAs
  // per SM) or when the block fills its 128 M rows anyway (256-row prefill chunks: measured 102 vs
  // 132 us per layer over 3,840 keys); the one with keys and head dims as M otherwise (its MMAs only
  // cover the real query rows).  The register-resident mma.sync kernel takes the other head sizes.
  // CS_ATTN_KERNEL=tc|tcw|mma, read when the context is created, forces one of them (tests run
  // them on the same inputs).
  int nsplit = 0;
  if (ctx->attn_force != 1) {
    const bool wide = ctx->attn_force == 3 || (ctx->attn_force == 0 && cs_attention_tc_tiles_per_cta(ctx, B, R) > 2 &&
                                               cs_attention_tc_group_rows(ctx, R) < 112);
    if (wide) nsplit = cs_launch_attention_tcw(ctx, kv_cache, layer, B, R, st);
    if (nsplit == 0) nsplit = cs_launch_attention_tc(ctx, kv_cache, layer, B, R, st);
  }
  if (nsplit > 0) {
    cs_launch_attn_merge(ctx, nsplit, B * R, st);
    return;
  }
  switch (ctx->cfg.head_dim) {
    case 32: nsplit = launch<32>(ctx, kv_cache, layer, B, R, st); break;
    case 64: nsplit = launch<64>(ctx, kv_cache, layer, B, R, st); break;
    default: nsplit = launch<128>(ctx, kv_cache, layer, B, R, st); break;
  }
  cs_launch_attn_merge(ctx, nsplit, B * R, st);
}
