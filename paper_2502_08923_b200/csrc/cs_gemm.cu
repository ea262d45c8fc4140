// Skinny bf16 projections of the verification forward (Sec. 3.2): Y = X W^T with at most
// 256 token rows and a large weight matrix that is streamed from HBM exactly once.
//
// The weight matrix is the M operand of the tensor-core instruction ("swap A/B"): one CTA
// owns 128 output features (UMMA M = 128) and all token rows (UMMA N = rows rounded up to
// 16), so even an 11-row block fills the 128 TMEM lanes.  Weights and activations arrive
// as TMA tiles of 64 K-elements (one 128-byte swizzled row per feature / token) through an
// mbarrier ring; one thread issues tcgen05.mma into a TMEM accumulator; four warps read
// it back with tcgen05.ld.  Activations are carried as two bf16 terms (x = hi + lo, lo being
// the rounding error of hi): both tiles are loaded and multiplied against the same weight
// tile, so the product is that of the fp32 activation although the operands are bf16.  The
// extra MMAs are free here: the kernel waits for weight bytes, not for the tensor pipe.
//
// K is split across the CTAs of a thread-block cluster (cluster dims (1, S, 1), S <= 8) so
// that every GEMM puts about two CTAs on each SM.  Each CTA leaves its partial tile in its
// own shared memory; after a cluster barrier every CTA sums one slice of the features over
// all ranks through distributed shared memory, in rank order (deterministic, no atomics,
// no partial sums in HBM), and applies the epilogue:
//   STORE     out[row][n]  = y                      (cs_linear)
//   QKV       rotates q and k (RoPE), writes q as the attention operand and appends the new
//             K/V rows to the bf16 cache            (QKV projection)
//   RESIDUAL  x[row][n]   += y                      (attention output and FFN down projections)
//   SWIGLU    act[row][j]  = bf16(silu(gate_j) * up_j), the tile holding 64 gate rows and the
//             64 matching up rows                   (FFN gate/up projection)
//   ARGMAX    per 128-feature tile (max logit, lowest token id) per row; logits are only
//             written when a debug buffer is given   (LM head)
//
// The kernel is launched with programmatic dependent launch: it starts while its
// predecessor drains, fills its pipeline with weight tiles (which depend on nothing) and
// only then waits for the predecessor before touching activations.
//
// Every wait is bounded: when it runs out the CTA records CS_DEV_TIMEOUT, drains its
// copies, still takes part in the cluster barriers, frees its TMEM and returns.
#include <stdlib.h>

#include <algorithm>
#include <type_traits>

#include "cs_common.cuh"

using std::max;
using std::min;

namespace {

constexpr int kThreads = 192;          // warps 0-3 epilogue, warp 4 TMA producer, warp 5 MMA
constexpr int kTileABytes = CS_GEMM_BM * CS_GEMM_BK * 2;   // 16 KB
constexpr unsigned long long kWaitLimitNs = 2000000000ull; // default limit of every wait: 2 s

struct GemmArgs {
  int rows, n_tok, N, K;
  int num_kb, kb_per_split, splits, stages, mode;
  float* out;            // STORE / RESIDUAL: [rows][N] fp32; ARGMAX: optional logits [rows][N]
  __nv_bfloat16* act;    // SWIGLU: [rows][F] bf16 (leading term)
  __nv_bfloat16* act_lo; // SWIGLU: second bf16 term of the same values, or NULL
  int lo_row;            // row coordinate of the activation operand's second bf16 term, -1 = none
  int F;
  QkvEpi q;              // QKV: where the rotated queries and the new K/V rows go
  NormFuse nf;           // RMSNorm folded into this GEMM's read-out (consumer) or residual update (producer)
  float* tile_max;       // ARGMAX: [rows][tile_stride] (a row's tile maxima are contiguous: the reduction reads them coalesced)
  int* tile_idx;
  int tile_stride;
  int* status;
  unsigned long long wait_ns;   // limit of every bounded wait
  int smem_bytes;               // dynamic shared memory of the launch
  int drop_kb;                  // test hook: the producer leaves out this K block's loads (-1 = none)
  unsigned long long* stamp;    // step timeline slot of this launch, or NULL
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when another role of this CTA gave up or `limit_ns` passed.
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                       unsigned long long limit_ns) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u) {
      if (*abort_flag) return false;
      const unsigned long long now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0,
                                            int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
// K-major operand tile, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);   // start address / 16
  d |= (uint64_t)1 << 16;                      // leading-dimension offset (unused here)
  d |= (uint64_t)(1024 >> 4) << 32;            // stride between 8-row groups / 16
  d |= (uint64_t)1 << 46;                      // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                      // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),
        "=r"(v[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  // the registers are valid only from here on: an empty statement that redefines them keeps their uses behind the wait
  asm volatile("" : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]), "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]) :: "memory");
}
// the two halves of the cluster barrier; like every barrier they count whole warps, so each
// warp executes each half exactly once, with all its lanes converged
__device__ __forceinline__ void cluster_arrive() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
  __syncwarp();
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %cluster_ctarank;" : "=r"(r));
  return r;
}
// Four consecutive floats of every rank's parked tile, summed in rank order.  All loads are
// issued before the first add so that their latencies overlap.
__device__ __forceinline__ float4 sum_over_ranks(uint32_t local_addr, int splits) {
  float4 v[CS_MAX_SPLITS];
#pragma unroll
  for (int q = 0; q < CS_MAX_SPLITS; ++q) {
    v[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q < splits) {
      uint32_t remote;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(q));
      asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                   : "=f"(v[q].x), "=f"(v[q].y), "=f"(v[q].z), "=f"(v[q].w)
                   : "r"(remote));
    }
  }
  float4 y = v[0];
#pragma unroll
  for (int q = 1; q < CS_MAX_SPLITS; ++q) { y.x += v[q].x; y.y += v[q].y; y.z += v[q].z; y.w += v[q].w; }
  return y;
}

// The remote loads behind two sums must have returned before what follows is issued: an
// empty asm that takes the sums as inputs cannot be scheduled before they exist.
__device__ __forceinline__ void keep_alive(const float4& p, const float4& q) {
  asm volatile("" ::"f"(p.x), "f"(p.y), "f"(p.z), "f"(p.w), "f"(q.x), "f"(q.y), "f"(q.z), "f"(q.w) : "memory");
}

// MT = 128-feature sub-tiles per CTA (compile-time, so that the one-tile kernel of the short blocks
// carries no loop overhead in its issue paths: its ring is latency-bound)
template <int MT>
__global__ void __launch_bounds__(kThreads, 1)
k_gemm_tc(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, GemmArgs a) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);   // operand tiles need 1024-byte alignment
  const int xtile = a.n_tok * 128;                 // one activation tile
  const bool two = a.lo_row >= 0;                   // activations come as two bf16 terms
  const int wbytes = MT * kTileABytes;            // the CTA's weight sub-tiles of one K block
  const int stage_bytes = wbytes + (two ? 2 : 1) * xtile;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)a.stages * stage_bytes);
  // bars[0..stages) = tile landed, bars[stages..2*stages) = tile consumed, bars[2*stages] = accumulator done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * a.stages + 1);
  volatile int* s_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_never = reinterpret_cast<volatile int*>(tmem_slot + 2);   // stays 0: drains wait on time only
  float* red_val = reinterpret_cast<float*>(tmem_slot + 4);       // [4][n_tok] (ARGMAX)
  int* red_idx = reinterpret_cast<int*>(red_val + 4 * a.n_tok);
  float* rstd_s = reinterpret_cast<float*>(red_idx + 4 * a.n_tok);   // [n_tok] (folded RMSNorm)
  float* dump = reinterpret_cast<float*>(smem);                   // [n_tok][128] fp32, reuses the operand ring
  // the launcher sizes the window for exactly this layout; a mismatch is reported, not written through
  if ((size_t)(reinterpret_cast<uint8_t*>(rstd_s + a.n_tok) - smem_raw) > (size_t)a.smem_bytes) {
    if (threadIdx.x == 0) atomicOr(a.status, CS_DEV_SMEM);
    return;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta_tile = blockIdx.x;
  const int split = (a.splits > 1) ? (int)cluster_rank() : 0;
  const int cta_n0 = cta_tile * MT * CS_GEMM_BM;
  const int kb0 = split * a.kb_per_split;
  const int kb1 = min(a.num_kb, kb0 + a.kb_per_split);
  const int nkb = max(0, kb1 - kb0);
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < MT * a.n_tok) tmem_cols <<= 1;   // one accumulator of n_tok columns per sub-tile

  const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + a.stages),
                 bar_acc = smem_u32(bars + 2 * a.stages);
  if (threadIdx.x == 128) {
    for (int s = 0; s < a.stages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    mbar_init(bar_acc, 1);
    *s_abort = 0;
    *s_never = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  bool ok = true;

  if (warp == 4) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      // weights depend on nothing: fill the ring with them before waiting for the predecessor
      const int npre = min(nkb, a.stages);
      for (int i = 0; i < npre; ++i) {
        if (i == a.drop_kb) continue;   // (test hook: this stage never fills, the consumer's wait runs out)
        mbar_expect_tx(bar_full + 8 * i, (uint32_t)stage_bytes);
#pragma unroll
        for (int m = 0; m < MT; ++m)
          tma_load_2d(smem_u32(smem + (size_t)i * stage_bytes) + m * kTileABytes, &tmW, bar_full + 8 * i,
                      (kb0 + i) * CS_GEMM_BK, cta_n0 + m * CS_GEMM_BM);
      }
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int i = 0; i < npre; ++i)
      {
        if (i == a.drop_kb) continue;
        const uint32_t sx = smem_u32(smem + (size_t)i * stage_bytes) + wbytes;
        tma_load_2d(sx, &tmX, bar_full + 8 * i, (kb0 + i) * CS_GEMM_BK, 0);
        if (two) tma_load_2d(sx + xtile, &tmX, bar_full + 8 * i, (kb0 + i) * CS_GEMM_BK, a.lo_row);
      }
      int i = npre;
      for (; i < nkb; ++i) {
        const int s = i % a.stages;
        const uint32_t ph = (uint32_t)(i / a.stages) & 1u;
        if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, s_abort, a.wait_ns)) { ok = false; break; }
        const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
        if (i == a.drop_kb) continue;
        mbar_expect_tx(bar_full + 8 * s, (uint32_t)stage_bytes);
#pragma unroll
        for (int m = 0; m < MT; ++m)
          tma_load_2d(sa + m * kTileABytes, &tmW, bar_full + 8 * s, (kb0 + i) * CS_GEMM_BK, cta_n0 + m * CS_GEMM_BM);
        tma_load_2d(sa + wbytes, &tmX, bar_full + 8 * s, (kb0 + i) * CS_GEMM_BK, 0);
        if (two) tma_load_2d(sa + wbytes + xtile, &tmX, bar_full + 8 * s, (kb0 + i) * CS_GEMM_BK, a.lo_row);
      }
      if (!ok) {
        *s_abort = 1;
        atomicOr(a.status, CS_DEV_TIMEOUT);
      }
      if (*s_abort) {
        // copies still in flight must land before this CTA's shared memory is reused or released
        for (int j = max(0, i - a.stages); j < i; ++j)
          if (j != a.drop_kb) mbar_wait(bar_full + 8 * (j % a.stages), (uint32_t)(j / a.stages) & 1u, s_never, a.wait_ns);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      // bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n_tok
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(a.n_tok >> 3) << 17) |
                             ((uint32_t)(CS_GEMM_BM >> 4) << 24);
      for (int i = 0; i < nkb; ++i) {
        const int s = i % a.stages;
        const uint32_t ph = (uint32_t)(i / a.stages) & 1u;
        if (!mbar_wait(bar_full + 8 * s, ph, s_abort, a.wait_ns)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
        const uint64_t db = umma_desc(sa + wbytes), dl = umma_desc(sa + wbytes + xtile);
#pragma unroll
        for (int m = 0; m < MT; ++m) {                   // every sub-tile against the same activation tile
          const uint64_t da = umma_desc(sa + m * kTileABytes);
          const uint32_t acc = tmem_base + (uint32_t)(m * a.n_tok);
#pragma unroll
          for (int kk = 0; kk < CS_GEMM_BK / 16; ++kk) {   // 16 K-elements = 32 bytes per instruction
            umma_bf16(acc, da + 2 * kk, db + 2 * kk, idesc, (i > 0 || kk > 0) ? 1u : 0u);
            if (two) umma_bf16(acc, da + 2 * kk, dl + 2 * kk, idesc, 1u);   // x = hi + lo
          }
        }
        umma_commit(bar_empty + 8 * s);
      }
      if (!ok) {
        *s_abort = 1;
        atomicOr(a.status, CS_DEV_TIMEOUT);
      }
      umma_commit(bar_acc);
    }
  } else {
    // ------------------------------------------------------------- epilogue warps 0-3: wait for the accumulators
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (a.nf.ssq_in != nullptr) {
      // 1/rms of every token row while the main loop runs: slots summed in a fixed order.  Eight
      // rows at a time, so that a tall block's loads overlap instead of queueing row after row.
      for (int tok0 = warp * 8; tok0 < a.rows; tok0 += 32) {
        float ss[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) ss[r] = 0.f;
        for (int sl = lane; sl < a.nf.slots_in; sl += 32) {
#pragma unroll
          for (int r = 0; r < 8; ++r)
            if (tok0 + r < a.rows) ss[r] += a.nf.ssq_in[(size_t)(tok0 + r) * a.nf.slot_stride + sl];
        }
#pragma unroll
        for (int r = 0; r < 8; ++r) {
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) ss[r] += __shfl_xor_sync(0xffffffffu, ss[r], off);
          if (lane == 0 && tok0 + r < a.rows) rstd_s[tok0 + r] = rsqrtf(ss[r] * a.nf.inv_d + a.nf.eps);
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
    }
    if (nkb > 0) ok = mbar_wait(bar_acc, 0, s_abort, a.wait_ns);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    ok = __all_sync(0xffffffffu, ok) && (*s_abort == 0);
    if (!ok && lane == 0) atomicOr(a.status, CS_DEV_TIMEOUT);
  }
  if (warp >= 4) asm volatile("griddepcontrol.wait;" ::: "memory");

  // One pass per 128-feature sub-tile: read its accumulator out, then (all but ARGMAX) the split-K
  // reduction and the epilogue.  Every CTA of a cluster takes the same number of passes.
#pragma unroll 1
  for (int m = 0; m < MT; ++m) {
  const int tile = cta_tile * MT + m;
  const int n0 = cta_n0 + m * CS_GEMM_BM;
  if (n0 >= a.N) break;
  if (warp < 4) {
    // ------------------------------------------------------------- accumulator read-out (warps 0-3)
    const int feat = n0 + warp * 32 + lane;
    const bool scaled = a.nf.ssq_in != nullptr;
    for (int c0 = 0; c0 < a.n_tok && c0 < a.rows; c0 += 16) {
      uint32_t v[16];
      if (nkb > 0 && ok) {
        tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(m * a.n_tok + c0), v);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = 0u;
      }
      if (scaled) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (c0 + j < a.rows) v[j] = __float_as_uint(__uint_as_float(v[j]) * rstd_s[c0 + j]);
      }
      if (a.mode != CS_EPI_ARGMAX) {
        // the MMAs have retired, so the operand ring is free: park the tile there
#pragma unroll
        for (int j = 0; j < 16; ++j) dump[(c0 + j) * CS_GEMM_BM + warp * 32 + lane] = __uint_as_float(v[j]);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int tok = c0 + j;
          float val = (feat < a.N) ? __uint_as_float(v[j]) : -INFINITY;
          int idx = feat;
          if (a.out != nullptr && tok < a.rows && feat < a.N) a.out[(size_t)tok * a.N + feat] = val;
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, val, off);
            const int oi = __shfl_xor_sync(0xffffffffu, idx, off);
            if (ov > val || (ov == val && oi < idx)) { val = ov; idx = oi; }
          }
          if (lane == 0) { red_val[warp * a.n_tok + tok] = val; red_idx[warp * a.n_tok + tok] = idx; }
        }
      }
    }
    if (a.mode == CS_EPI_ARGMAX) {
      asm volatile("bar.sync 1, 128;" ::: "memory");   // the four epilogue warps only
      if (ok) {
        for (int tok = threadIdx.x; tok < a.rows; tok += 128) {
          float val = red_val[tok];
          int idx = red_idx[tok];
#pragma unroll
          for (int w = 1; w < 4; ++w) {
            const float ov = red_val[w * a.n_tok + tok];
            const int oi = red_idx[w * a.n_tok + tok];
            if (ov > val || (ov == val && oi < idx)) { val = ov; idx = oi; }
          }
          a.tile_max[(size_t)tok * a.tile_stride + tile] = val;
          a.tile_idx[(size_t)tok * a.tile_stride + tile] = idx;
        }
      }
      if (MT > 1) asm volatile("bar.sync 1, 128;" ::: "memory");   // the scratch rows are reused by the next pass
    }
  }

  // ---------------------------------------------------------------- split-K reduction + epilogue
  if (a.mode != CS_EPI_ARGMAX) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    // Cluster barrier 1: every rank's tile is parked.  Barrier 2 (nobody leaves while a peer
    // still reads its tile) is split: a warp arrives as soon as the last remote reads of its lanes
    // have returned and only waits after its global stores, which hides the barrier behind them.
    if (a.splits > 1) cluster_arrive();
    const int e = threadIdx.x;
    // residual update: the first item's x (and gain) can be on their way during the barrier
    const int r_fs = ((CS_GEMM_BM + a.splits - 1) / a.splits + 3) & ~3;
    const int r_flo = split * r_fs, r_per_tok = max(0, min(CS_GEMM_BM, r_flo + r_fs) - r_flo) >> 2;
    const bool r_vec = (a.N & 3) == 0;
    float4 x_pre = make_float4(0.f, 0.f, 0.f, 0.f);
    if (warp < 4 && a.mode == CS_EPI_RESIDUAL && r_vec && e < r_per_tok * a.rows) {
      const int f = r_flo + 4 * (e % r_per_tok), tok = e / r_per_tok;
      if (n0 + f + 3 < a.N) x_pre = *reinterpret_cast<const float4*>(a.out + (size_t)tok * a.N + n0 + f);
    }
    if (a.splits > 1) cluster_wait();
    bool arrived = a.splits <= 1;                  // this thread's half of barrier 2
    if (warp < 4) {
      const uint32_t dump_addr = smem_u32(dump);
      if (a.mode == CS_EPI_QKV) {
        // RoPE pairs feature i of a head with i + Dh/2: both lie in this tile.  j in [0,64) walks
        // the first halves of the tile's heads; each rank finishes a slice of j, four at a time.
        const QkvEpi& Q = a.q;
        const int half = Q.Dh >> 1;
        const int js = ((64 + a.splits - 1) / a.splits + 3) & ~3;
        const int j_lo = split * js, j_n = max(0, min(64, j_lo + js) - j_lo);
        const int per_tok = j_n >> 2;
        const int total = per_tok * a.rows, iters = (total + 127) >> 7;   // same trip count for every thread
        for (int it = 0; it < iters; ++it) {
          const int idx = e + (it << 7);
          const int idc = idx < total ? idx : 0;
          const int j = j_lo + 4 * (idc % per_tok), tok = idc / per_tok;
          const int i = j % half, f1 = (j / half) * Q.Dh + i, f2 = f1 + half;
          const int head = (n0 + f1) / Q.Dh;
          const bool act = idx < total && head < Q.H + 2 * Q.Hkv;
          // the rotation factors and the row's place in the cache do not depend on the sums: they are
          // requested first, so that their latency runs under the remote reads
          const float4* csp = reinterpret_cast<const float4*>(Q.rope_cs + 2 * ((size_t)tok * half + i));
          const float4 cs01 = csp[0], cs23 = csp[1];      // (cos, sin) of dims i .. i + 3
          const int row_w = Q.row_write[tok], row_p = Q.row_pos[tok];
          float4 av = make_float4(0.f, 0.f, 0.f, 0.f), bv = av;
          if (a.splits > 1) {
            if (act) {
              av = sum_over_ranks(dump_addr + 4u * (uint32_t)(tok * CS_GEMM_BM + f1), a.splits);
              bv = sum_over_ranks(dump_addr + 4u * (uint32_t)(tok * CS_GEMM_BM + f2), a.splits);
            }
            if (it == iters - 1) { keep_alive(av, bv); cluster_arrive(); arrived = true; }
          } else if (act) {
            av = *reinterpret_cast<const float4*>(dump + tok * CS_GEMM_BM + f1);
            bv = *reinterpret_cast<const float4*>(dump + tok * CS_GEMM_BM + f2);
          }
          if (!act) continue;
          const float a4[4] = {av.x, av.y, av.z, av.w}, b4[4] = {bv.x, bv.y, bv.z, bv.w};
          float r0[4], r1[4];
          const bool is_v = head >= Q.H + Q.Hkv;
          const float2 csv[4] = {make_float2(cs01.x, cs01.y), make_float2(cs01.z, cs01.w), make_float2(cs23.x, cs23.y), make_float2(cs23.z, cs23.w)};
#pragma unroll
          for (int t4 = 0; t4 < 4; ++t4) {
            const float2 cs2 = csv[t4];
            r0[t4] = is_v ? a4[t4] : a4[t4] * cs2.x - b4[t4] * cs2.y;
            r1[t4] = is_v ? b4[t4] : b4[t4] * cs2.x + a4[t4] * cs2.y;
          }
          __nv_bfloat162 h0[2], h1[2];
          h0[0] = __floats2bfloat162_rn(r0[0], r0[1]); h0[1] = __floats2bfloat162_rn(r0[2], r0[3]);
          h1[0] = __floats2bfloat162_rn(r1[0], r1[1]); h1[1] = __floats2bfloat162_rn(r1[2], r1[3]);
          if (head < Q.H) {
            // rotated query as two bf16 terms, the attention kernel's operand
            __nv_bfloat16* qd = Q.qbuf + ((size_t)tok * Q.H + head) * Q.Dh + i;
            __nv_bfloat16* ql = qd + (size_t)CS_MAX_ROWS * Q.H * Q.Dh;
            *reinterpret_cast<uint2*>(qd) = *reinterpret_cast<const uint2*>(h0);
            *reinterpret_cast<uint2*>(qd + half) = *reinterpret_cast<const uint2*>(h1);
            const float2 f00 = __bfloat1622float2(h0[0]), f01 = __bfloat1622float2(h0[1]);
            const float2 f10 = __bfloat1622float2(h1[0]), f11 = __bfloat1622float2(h1[1]);
            __nv_bfloat162 l0[2], l1[2];
            l0[0] = __floats2bfloat162_rn(r0[0] - f00.x, r0[1] - f00.y); l0[1] = __floats2bfloat162_rn(r0[2] - f01.x, r0[3] - f01.y);
            l1[0] = __floats2bfloat162_rn(r1[0] - f10.x, r1[1] - f10.y); l1[1] = __floats2bfloat162_rn(r1[2] - f11.x, r1[3] - f11.y);
            *reinterpret_cast<uint2*>(ql) = *reinterpret_cast<const uint2*>(l0);
            *reinterpret_cast<uint2*>(ql + half) = *reinterpret_cast<const uint2*>(l1);
          } else if (row_w) {
            // new K (rotated) / V row of the cache, stored in bf16
            const int kvh = is_v ? head - Q.H - Q.Hkv : head - Q.H;
            __nv_bfloat16* dst = Q.kv + ((((size_t)Q.layer * 2 + (is_v ? 1 : 0)) * Q.max_batch + tok / Q.R) * Q.Hkv + kvh) *
                                            (size_t)Q.max_seq * Q.Dh + (size_t)row_p * Q.Dh + i;
            *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(h0);
            *reinterpret_cast<uint2*>(dst + half) = *reinterpret_cast<const uint2*>(h1);
          }
        }
      } else if (a.mode == CS_EPI_SWIGLU) {
        // features 0..63 of the tile are gate rows, 64..127 the matching up rows; each rank
        // finishes a slice of j (a multiple of 4 wide), four consecutive j per thread
        const int js = ((64 + a.splits - 1) / a.splits + 3) & ~3;
        const int j_lo = split * js, j_n = max(0, min(64, j_lo + js) - j_lo);
        const int per_tok = j_n >> 2;
        const int total = per_tok * a.rows, iters = (total + 127) >> 7;
        for (int it = 0; it < iters; ++it) {
          const int idx = e + (it << 7);
          const bool act = idx < total;
          const int idc = act ? idx : 0;
          const int j = j_lo + 4 * (idc % per_tok), tok = idc / per_tok;
          float4 g = make_float4(0.f, 0.f, 0.f, 0.f), u = g;
          if (a.splits > 1) {
            if (act) {
              g = sum_over_ranks(dump_addr + 4u * (uint32_t)(tok * CS_GEMM_BM + j), a.splits);
              u = sum_over_ranks(dump_addr + 4u * (uint32_t)(tok * CS_GEMM_BM + 64 + j), a.splits);
            }
            if (it == iters - 1) { keep_alive(g, u); cluster_arrive(); arrived = true; }
          } else if (act) {
            g = *reinterpret_cast<const float4*>(dump + tok * CS_GEMM_BM + j);
            u = *reinterpret_cast<const float4*>(dump + tok * CS_GEMM_BM + 64 + j);
          }
          if (!act) continue;
          const float gv[4] = {g.x, g.y, g.z, g.w}, uv[4] = {u.x, u.y, u.z, u.w};
          const int jj0 = tile * 64 + j;
          if ((a.F & 3) == 0 && jj0 + 3 < a.F) {
            float v4[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) v4[i] = __fdividef(gv[i], 1.f + __expf(-gv[i])) * uv[i];
            __nv_bfloat162 h[2], l[2];
            h[0] = __floats2bfloat162_rn(v4[0], v4[1]); h[1] = __floats2bfloat162_rn(v4[2], v4[3]);
            const float2 h0 = __bfloat1622float2(h[0]), h1 = __bfloat1622float2(h[1]);
            l[0] = __floats2bfloat162_rn(v4[0] - h0.x, v4[1] - h0.y); l[1] = __floats2bfloat162_rn(v4[2] - h1.x, v4[3] - h1.y);
            *reinterpret_cast<uint2*>(a.act + (size_t)tok * a.F + jj0) = *reinterpret_cast<const uint2*>(h);
            if (a.act_lo != nullptr) *reinterpret_cast<uint2*>(a.act_lo + (size_t)tok * a.F + jj0) = *reinterpret_cast<const uint2*>(l);
            continue;
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int jj = tile * 64 + j + i;
            if (jj < a.F) {
              const float v = __fdividef(gv[i], 1.f + __expf(-gv[i])) * uv[i];
              const __nv_bfloat16 hi = __float2bfloat16_rn(v);
              a.act[(size_t)tok * a.F + jj] = hi;
              if (a.act_lo != nullptr) a.act_lo[(size_t)tok * a.F + jj] = __float2bfloat16_rn(v - __bfloat162float(hi));
            }
          }
        }
      } else {
        const int fs = ((CS_GEMM_BM + a.splits - 1) / a.splits + 3) & ~3;
        const int f_lo = split * fs, f_n = max(0, min(CS_GEMM_BM, f_lo + fs) - f_lo);
        const int per_tok = f_n >> 2;
        const bool feeds_norm = a.mode == CS_EPI_RESIDUAL && a.nf.gain_out != nullptr;
        float* part = dump + a.n_tok * CS_GEMM_BM;   // [rows][32] sums of squares, behind the parked tile
        const int total = per_tok * a.rows, iters = (total + 127) >> 7;
        const bool vec_n = (a.N & 3) == 0;
        // Tall blocks take two items per turn: the remote reads and the residual reads of both are
        // requested before either is finished, so a dozen turns per thread overlap pairwise (128
        // threads on an otherwise idle SM have nothing else to hide those latencies behind).  Short
        // blocks have one turn and take it without the second item's bookkeeping.
        auto turns = [&](auto per_turn) {
        constexpr int NU = decltype(per_turn)::value;
        for (int it = 0; it < iters; it += NU) {
          int idx[NU], f[NU], tok[NU];
          bool act[NU], vec[NU];
          float4 y[NU], x[NU];
#pragma unroll
          for (int u = 0; u < NU; ++u) {
            idx[u] = e + ((it + u) << 7);
            act[u] = it + u < iters && idx[u] < total;
            const int idc = act[u] ? idx[u] : 0;
            f[u] = f_lo + 4 * (idc % per_tok);
            tok[u] = idc / per_tok;
            vec[u] = vec_n && n0 + f[u] + 3 < a.N;
            y[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            x[u] = y[u];
          }
          if (a.splits > 1) {
#pragma unroll
            for (int u = 0; u < NU; ++u)
              if (act[u]) y[u] = sum_over_ranks(dump_addr + 4u * (uint32_t)(tok[u] * CS_GEMM_BM + f[u]), a.splits);
          } else {
#pragma unroll
            for (int u = 0; u < NU; ++u)
              if (act[u]) y[u] = *reinterpret_cast<const float4*>(dump + tok[u] * CS_GEMM_BM + f[u]);
          }
          if (a.mode == CS_EPI_RESIDUAL) {
#pragma unroll
            for (int u = 0; u < NU; ++u)
              if (act[u] && vec[u])
                x[u] = (it + u == 0) ? x_pre : *reinterpret_cast<const float4*>(a.out + (size_t)tok[u] * a.N + n0 + f[u]);
          }
          if (a.splits > 1 && it + NU >= iters) { keep_alive(y[0], y[NU - 1]); cluster_arrive(); arrived = true; }
#pragma unroll
          for (int u = 0; u < NU; ++u) {
            if (!act[u]) continue;
            if (feeds_norm) part[tok[u] * 32 + idx[u] % per_tok] = 0.f;
            float* dst = a.out + (size_t)tok[u] * a.N + n0 + f[u];
            if (vec[u]) {
              float4 o = y[u];
              o.x += x[u].x; o.y += x[u].y; o.z += x[u].z; o.w += x[u].w;   // (x stays 0 unless this is a residual update)
              *reinterpret_cast<float4*>(dst) = o;
              if (feeds_norm) {
                const uint2 gw = *reinterpret_cast<const uint2*>(a.nf.gain_out + n0 + f[u]);
                const float2 g01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw.x));
                const float2 g23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw.y));
                const float w0 = o.x * g01.x, w1 = o.y * g01.y, w2 = o.z * g23.x, w3 = o.w * g23.y;
                __nv_bfloat162 h[2], l[2];
                h[0] = __floats2bfloat162_rn(w0, w1); h[1] = __floats2bfloat162_rn(w2, w3);
                const float2 h0 = __bfloat1622float2(h[0]), h1 = __bfloat1622float2(h[1]);
                l[0] = __floats2bfloat162_rn(w0 - h0.x, w1 - h0.y); l[1] = __floats2bfloat162_rn(w2 - h1.x, w3 - h1.y);
                __nv_bfloat16* xo = a.nf.xn_out + (size_t)tok[u] * a.N + n0 + f[u];
                *reinterpret_cast<uint2*>(xo) = *reinterpret_cast<const uint2*>(h);
                *reinterpret_cast<uint2*>(xo + (size_t)CS_MAX_ROWS * a.N) = *reinterpret_cast<const uint2*>(l);
                part[tok[u] * 32 + idx[u] % per_tok] = (o.x * o.x + o.y * o.y) + (o.z * o.z + o.w * o.w);
              }
            } else {
              const float yv[4] = {y[u].x, y[u].y, y[u].z, y[u].w};
#pragma unroll
              for (int i = 0; i < 4; ++i)
                if (n0 + f[u] + i < a.N) dst[i] = (a.mode == CS_EPI_RESIDUAL) ? dst[i] + yv[i] : yv[i];
            }
          }
        }
        };
        if (iters > 1) turns(std::integral_constant<int, 2>{});
        else turns(std::integral_constant<int, 1>{});
        if (feeds_norm) {
          asm volatile("bar.sync 1, 128;" ::: "memory");
          for (int tok = e; tok < a.rows; tok += 128) {
            float ss = 0.f;
            for (int q = 0; q < per_tok; ++q) ss += part[tok * 32 + q];
            a.nf.ssq_out[(size_t)tok * a.nf.slot_stride + tile * a.splits + split] = ss;
          }
        }
      }
    }
    if (a.splits > 1) {
      if (!arrived) cluster_arrive();
      cluster_wait();                              // nobody leaves (or parks its next tile) while a peer still reads this one
    } else if (MT > 1) {
      __syncthreads();                             // the parked tile is read out before the next one is parked
    }
  }
  }   // sub-tile passes
  // ---------------------------------------------------------------- teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (threadIdx.x == 0) cs_stamp_end(a.stamp);
  if (warp == 5) {
    if (*s_abort && lane == 0 && nkb > 0) mbar_wait(bar_acc, 0, s_never, a.wait_ns);  // MMAs retired
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols)
                 : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [rows][K] bf16 row-major, tiles of box_rows x 64 elements, 128-byte swizzle, zero fill
cs_status encode_2d(cs_ctx* ctx, CUtensorMap* tm, const void* base, int rows, int K, int box_rows,
                    bool weights) {
  EncodeTiledFn enc = get_encode();
  if (enc == nullptr) {
    snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled is not available");
    return CS_ERR_CUDA;
  }
  if ((reinterpret_cast<uintptr_t>(base) & 15) != 0 || (K % 8) != 0) {
    snprintf(ctx->err, sizeof(ctx->err), "operand needs a 16-byte aligned base and K %% 8 == 0");
    return CS_ERR_SHAPE;
  }
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {(cuuint32_t)CS_GEMM_BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   weights ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled failed with %d (rows %d, K %d, box %d)",
             (int)r, rows, K, box_rows);
    return CS_ERR_CUDA;
  }
  return CS_OK;
}

}  // namespace

cs_status cs_encode_tiled(cs_ctx* ctx, CUtensorMap* tm, const void* base, int rank, const unsigned long long* dims,
                          const unsigned long long* strides_bytes, const unsigned* box) {
  EncodeTiledFn enc = get_encode();
  if (enc == nullptr) {
    snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled is not available");
    return CS_ERR_CUDA;
  }
  if (rank < 1 || rank > 5 || (reinterpret_cast<uintptr_t>(base) & 15) != 0) {
    snprintf(ctx->err, sizeof(ctx->err), "tensor map needs rank 1..5 and a 16-byte aligned base");
    return CS_ERR_SHAPE;
  }
  cuuint64_t d[5], sb[4];
  cuuint32_t bx[5], estr[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; estr[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) sb[i] = strides_bytes[i];
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, sb, bx, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->err, sizeof(ctx->err), "cuTensorMapEncodeTiled (rank %d) failed with %d", rank, (int)r);
    return CS_ERR_CUDA;
  }
  return CS_OK;
}

cs_status cs_gemm_plan(cs_ctx* ctx, GemmPlan* g, const void* w, int N, int K, bool allow_split) {
  g->W = static_cast<const __nv_bfloat16*>(w);
  g->N = N;
  g->K = K;
  g->allow_split = allow_split;
  const int tiles = cs_ceil_div(N, CS_GEMM_BM), kb = cs_ceil_div(K, CS_GEMM_BK);
  // two CTAs fit on an SM; clustered launches are planned for 85 % of those slots, because
  // a cluster must find all its CTAs free inside one GPC and a grid that needs every slot
  // spills into a second wave
  const int slots = 2 * ctx->num_sms;
  int best = 1;
  long best_cost = -1;
  const int smax = allow_split ? cs_max_splits(tiles, kb) : 1;
  for (int s = 1; s <= smax; ++s) {
    const int avail = (s > 1) ? slots * 85 / 100 : slots;
    // waves of CTAs times the K blocks each CTA streams, plus a fixed start-up/epilogue cost
    const long cost = (long)cs_ceil_div(tiles * s, avail) * (cs_ceil_div(kb, s) + 2);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
  }
  g->kb_per_split = cs_ceil_div(kb, best);
  g->splits = cs_ceil_div(kb, g->kb_per_split);
  return encode_2d(ctx, &g->tmW, w, N, K, CS_GEMM_BM, true);
}

static cs_status ensure_gemm_attrs(cs_ctx* ctx) {
  if (!ctx->gemm_attr_set) {
    CS_CUDA_OK(ctx, cudaFuncSetAttribute(k_gemm_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    CS_CUDA_OK(ctx, cudaFuncSetAttribute(k_gemm_tc<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    CS_CUDA_OK(ctx, cudaFuncSetAttribute(k_gemm_tc<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    ctx->gemm_attr_set = true;
  }
  return CS_OK;
}

// How many clusters of `spl` one-CTA-per-SM CTAs the device runs at once.  A cluster has to find
// all its CTAs inside one GPC, so this can be well below SMs / spl: 48 clusters of 3 do not fit
// on 148 SMs, and a launch that needs them takes two waves.  Asked of the runtime once per shape.
static int tall_clusters_at_once(const cs_ctx* cctx, int mt, int spl, int smem) {
  cs_ctx* ctx = const_cast<cs_ctx*>(cctx);
  if (spl <= 1) return ctx->num_sms;
  int& slot = ctx->tall_clusters[mt == 4 ? 2 : (mt == 2 ? 1 : 0)][spl];
  if (slot == 0) {
    int n = 0;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(ctx->num_sms, spl, 1);
    lc.blockDim = dim3(kThreads, 1, 1);
    lc.dynamicSmemBytes = (size_t)smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = spl; at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    void (*kernel)(const CUtensorMap, const CUtensorMap, GemmArgs) = mt == 4 ? k_gemm_tc<4> : (mt == 2 ? k_gemm_tc<2> : k_gemm_tc<1>);
    if (ensure_gemm_attrs(ctx) == CS_OK && cudaOccupancyMaxActiveClusters(&n, kernel, &lc) == cudaSuccess && n > 0) slot = n;
    else { (void)cudaGetLastError(); slot = max(1, ctx->num_sms * 85 / 100 / spl); }   // no answer: the planner's allowance
  }
  return slot;
}

// Launch shape of one GEMM for a block of `rows` token rows.
//  - Short blocks (two CTAs fit on an SM): one 128-feature tile per CTA and the plan's split-K
//    factor, made for two CTAs per SM - the HBM-bound regime of 11-row blocks.
//  - Tall blocks (one CTA per SM): every CTA re-reads its K range of the activations from L2,
//    which at 100+ rows is several times the weight bytes, so a CTA takes 2 or 4 sub-tiles that
//    share each activation tile (one TMEM accumulator each), and the split-K factor is chosen
//    for whole waves of one CTA per SM.  Candidates are ranked by a cost model calibrated on
//    measurements (K blocks per CTA times the cost of one, plus the epilogue, times waves).
cs_status cs_gemm_shape(const cs_ctx* ctx, const GemmPlan* g, int rows, bool two_terms, GemmShape* out) {
  GemmShape sh = {};
  sh.n_tok = cs_ceil_div(rows, 16) * 16;
  const int terms = two_terms ? 2 : 1;
  const int xbytes = terms * sh.n_tok * 128;
  const int tiles = cs_ceil_div(g->N, CS_GEMM_BM), kb = cs_ceil_div(g->K, CS_GEMM_BK);
  // behind the ring: up to 2 * 8 + 1 barriers, the TMEM slot and flags, the ARGMAX scratch and 1/rms
  const int fixed = 1024 /*alignment slack*/ + (2 * 8 + 1) * 8 + 16 + 9 * sh.n_tok * 4;
  const size_t park = (size_t)sh.n_tok * (CS_GEMM_BM + 32) * 4;   // parked tile + sums of squares reuse the ring
  const int sb1 = kTileABytes + xbytes;
  // Two CTAs per SM wherever two stages fit into half an SM: the grids (224-240 CTAs) are
  // sized for the 296 slots that gives.  Only blocks too tall for that take the whole SM.
  int stages = (100 * 1024 - fixed) / sb1;
  bool tall = false;
  if (stages < 4) {
    const int two = (113 * 1024 - fixed) / sb1;
    if (two >= 2 && (size_t)two * sb1 >= park) stages = two;
    else tall = true;
  }
  if (!tall) {
    sh.mt = 1;
    sh.stages = stages > 8 ? 8 : stages;
    sh.splits = g->splits;
    sh.kb_per_split = g->kb_per_split;
    sh.stage_bytes = sb1;
  } else {
    long best = -1;
    for (int mt = 1; mt <= 4; mt *= 2) {
      if (mt * sh.n_tok > 512 || (mt > 1 && mt > tiles)) continue;
      const int sb = mt * kTileABytes + xbytes;
      int st = (220 * 1024 - fixed) / sb;
      if (st > 8) st = 8;
      if (st < 2 || (size_t)st * sb < park) continue;
      const int ctas = cs_ceil_div(tiles, mt);
      // Cycles of one K block, calibrated on 176-row blocks: the mt * terms * 4 MMAs take n_tok / 2
      // cycles each; a stage comes back L cycles after it was handed to the producer (about 2,100
      // for a 61 KB stage, 3,300 for a 77 KB one), and with `st` stages in flight a K block costs
      // (L + mma) / st unless the tensor pipe is the slower.  The epilogue (accumulator read-out,
      // split-K reduction over the cluster, stores) costs about 4,000 + 145 n_tok cycles per sub-tile.
      const long mma = (long)mt * terms * 4 * (sh.n_tok / 2);
      const long lat = 2120 + (long)((sb - 62464) * 0.072);
      const long turn = ((lat > 1000 ? lat : 1000) + mma) / st;
      const long per_kb = mma > turn ? mma : turn;
      const long epi = (long)mt * (4000 + 145L * sh.n_tok);
      const int smax = g->allow_split ? max(1, min(CS_MAX_SPLITS, kb / 4)) : 1;
      for (int sp = 1; sp <= smax; ++sp) {
        const int kps = cs_ceil_div(kb, sp), spl = cs_ceil_div(kb, kps);
        const long waves = cs_ceil_div(ctas, tall_clusters_at_once(ctx, mt, spl, fixed + st * sb));
        const long cost = waves * ((long)kps * per_kb + epi);
        if (best < 0 || cost < best) {
          best = cost;
          sh.mt = mt; sh.stages = st; sh.splits = spl; sh.kb_per_split = kps; sh.stage_bytes = sb;
        }
      }
    }
    if (best < 0) return CS_ERR_UNSUPPORTED;
  }
  if (sh.stages < 2 || (size_t)sh.stages * sh.stage_bytes < park) return CS_ERR_UNSUPPORTED;
  sh.smem = fixed + sh.stages * sh.stage_bytes;
  *out = sh;
  return CS_OK;
}

cs_status cs_make_act_map(cs_ctx* ctx, CUtensorMap* tm, const void* base, int rows_total, int K,
                          int box_rows) {
  return encode_2d(ctx, tm, base, rows_total, K, box_rows, false);
}

cs_status cs_launch_gemm(cs_ctx* ctx, const GemmPlan* g, const CUtensorMap* tmX, int lo_row, int rows, int mode,
                         float* out, __nv_bfloat16* act, __nv_bfloat16* act_lo, int F, const QkvEpi* q,
                         const NormFuse* nf, cudaStream_t st) {
  GemmShape sh;
  if (cs_gemm_shape(ctx, g, rows, lo_row >= 0, &sh) != CS_OK) {
    snprintf(ctx->err, sizeof(ctx->err), "no GEMM launch shape fits shared memory for %d rows", rows);
    return CS_ERR_UNSUPPORTED;
  }
  const int tiles = cs_ceil_div(cs_ceil_div(g->N, CS_GEMM_BM), sh.mt);   // CTAs along the features
  GemmArgs a;
  a.rows = rows;
  a.n_tok = sh.n_tok;
  a.N = g->N;
  a.K = g->K;
  a.num_kb = cs_ceil_div(g->K, CS_GEMM_BK);
  a.splits = sh.splits;
  a.kb_per_split = sh.kb_per_split;
  a.mode = mode;
  a.out = out;
  a.act = act;
  a.act_lo = act_lo;
  a.lo_row = lo_row;
  a.F = F;
  if (q != nullptr) a.q = *q;
  a.nf = NormFuse{};
  if (nf != nullptr) a.nf = *nf;
  if (a.nf.gain_out != nullptr && (mode != CS_EPI_RESIDUAL || (g->N & 3) != 0)) {
    snprintf(ctx->err, sizeof(ctx->err), "a norm can only be folded into a residual GEMM whose width is a multiple of 4");
    return CS_ERR_UNSUPPORTED;
  }
  a.tile_max = ctx->tile_max;
  a.tile_idx = ctx->tile_idx;
  a.tile_stride = cs_ceil_div(g->N, CS_GEMM_BM);
  a.status = ctx->d_status;
  a.stages = sh.stages;
  const size_t smem = (size_t)sh.smem;
  a.smem_bytes = sh.smem;
  a.wait_ns = ctx->wait_limit_ns;
  a.stamp = cs_next_stamp(ctx, mode == CS_EPI_ARGMAX ? CS_FAM_LMHEAD : CS_FAM_GEMM);
  a.drop_kb = ctx->debug_drop_kb;
  ctx->debug_drop_kb = -1;            // the hook covers one launch
  if (a.drop_kb >= 0 && a.splits > 1) {
    snprintf(ctx->err, sizeof(ctx->err), "the dropped-tile test hook is for launches without split-K");
    return CS_ERR_UNSUPPORTED;
  }
  void (*kernel)(const CUtensorMap, const CUtensorMap, GemmArgs) =
      sh.mt == 4 ? k_gemm_tc<4> : (sh.mt == 2 ? k_gemm_tc<2> : k_gemm_tc<1>);
  {
    const cs_status as = ensure_gemm_attrs(ctx);
    if (as != CS_OK) return as;
  }
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(tiles, a.splits, 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute at[2];
  int na = 0;
  at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[na].val.programmaticStreamSerializationAllowed = 1;
  ++na;
  if (a.splits > 1) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = 1;
    at[na].val.clusterDim.y = a.splits;
    at[na].val.clusterDim.z = 1;
    ++na;
  }
  lc.attrs = at;
  lc.numAttrs = na;
  CS_CUDA_OK(ctx, cudaLaunchKernelEx(&lc, kernel, g->tmW, *tmX, a));
  return CS_OK;
}

// ------------------------------------------------------------------------------------------
// cs_lm_head_static: the LM-head argmax stage for callers that may not allocate.
//
// The tile-argmax epilogue above needs somewhere to put one (max logit, token id) pair per
// 128-token-id tile and row before the final reduction.  Every other entry point takes that
// room from the workspace the caller allocated for cs_create.  This one takes it from a fixed
// array that is part of the library image, so a caller that cannot obtain device memory of
// its own at that moment (inside a memory-pool callback, in a plug-in that is handed input and
// output buffers but no allocator, late in a process whose memory is fully committed) can
// still ask for greedy tokens.  The price: a fixed maximum size, 512 KB held on every GPU
// that loads the library until the process exits, and one array shared by all calls.
namespace {

constexpr int kStaticMaxRows = 64;                       // rows per call
constexpr int kStaticMaxTiles = 1024;                    // 128-id tiles: vocab <= 131072
constexpr size_t kStaticMaxBytes = (size_t)kStaticMaxTiles * kStaticMaxRows * 4;
// [tile maxima fp32][tile ids int32][status word + padding]
static __device__ __align__(256) unsigned char g_lm_scratch[2 * kStaticMaxBytes + 256];

// Host code must not pass `g_lm_scratch` itself to a kernel: on the host that name is only a
// handle for the runtime.  The device address is looked up once per device and kept here.
constexpr int kMaxDevices = 64;
void* g_lm_scratch_dev[kMaxDevices] = {nullptr};

cs_status static_scratch(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CS_ERR_CUDA;
  if (g_lm_scratch_dev[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_lm_scratch) != cudaSuccess || p == nullptr) return CS_ERR_CUDA;
    if (cudaFuncSetAttribute(k_gemm_tc<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
      return CS_ERR_CUDA;
    g_lm_scratch_dev[dev] = p;
  }
  *out = g_lm_scratch_dev[dev];
  return CS_OK;
}

// greedy token per row from the per-tile pairs; -2 marks a row whose GEMM gave up on a wait
__global__ void __launch_bounds__(128)
k_tile_reduce_static(const float* __restrict__ tile_max, const int* __restrict__ tile_idx, int tiles,
                     int tile_stride, const int* __restrict__ status, int* __restrict__ ids) {
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
    ids[row] = (*status != 0) ? -2 : ((idx == INT32_MAX) ? -1 : idx);
  }
}

}  // namespace

extern "C" cs_status cs_lm_head_static(const void* X, const void* W, int rows, int vocab, int d_model,
                                       int32_t* ids, void* stream) {
  if (X == nullptr || W == nullptr || ids == nullptr || rows < 1 || vocab < 1 || d_model < 8 || (d_model % 8))
    return CS_ERR_ARG;
  if (((reinterpret_cast<uintptr_t>(X) | reinterpret_cast<uintptr_t>(W)) & 15) != 0) return CS_ERR_ARG;
  const int tiles = cs_ceil_div(vocab, CS_GEMM_BM);
  if (rows > kStaticMaxRows || tiles > kStaticMaxTiles) return CS_ERR_LIMIT;
  void* scratch = nullptr;
  cs_status s = static_scratch(&scratch);
  if (s != CS_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* tile_max = static_cast<float*>(scratch);
  int* tile_idx = reinterpret_cast<int*>(static_cast<unsigned char*>(scratch) + kStaticMaxBytes);
  int* status = reinterpret_cast<int*>(static_cast<unsigned char*>(scratch) + 2 * kStaticMaxBytes);

  // host work that can fail comes first, so that a failed call has enqueued nothing
  cs_ctx err_sink;                      // only its error string is touched by the encoder
  err_sink.err[0] = 0;
  CUtensorMap tmW, tmX;
  GemmArgs a;
  a.rows = rows;
  a.n_tok = cs_ceil_div(rows, 16) * 16;
  if (encode_2d(&err_sink, &tmW, W, vocab, d_model, CS_GEMM_BM, true) != CS_OK) return CS_ERR_CUDA;
  if (encode_2d(&err_sink, &tmX, X, a.n_tok, d_model, a.n_tok, false) != CS_OK) return CS_ERR_CUDA;
  // the array keeps whatever the last call left: the status word is the only part that is
  // read before it is written, so it is the only part cleared
  if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return CS_ERR_CUDA;
  a.N = vocab;
  a.K = d_model;
  a.num_kb = cs_ceil_div(d_model, CS_GEMM_BK);
  a.kb_per_split = a.num_kb;
  a.splits = 1;
  a.mode = CS_EPI_ARGMAX;
  a.out = nullptr;
  a.act = nullptr;
  a.act_lo = nullptr;
  a.lo_row = -1;
  a.F = 0;
  a.nf = NormFuse{};
  a.tile_max = tile_max;
  a.tile_idx = tile_idx;
  a.tile_stride = kStaticMaxTiles;
  a.status = status;
  const int stage_bytes = kTileABytes + a.n_tok * 128;
  const int fixed = 1024 + (2 * 8 + 1) * 8 + 16 + 9 * a.n_tok * 4;
  int stages = (100 * 1024 - fixed) / stage_bytes;   // at least 4 for rows <= 64
  if (stages > 8) stages = 8;
  a.stages = stages;
  a.smem_bytes = fixed + stages * stage_bytes;
  a.wait_ns = kWaitLimitNs;
  a.drop_kb = -1;
  a.stamp = nullptr;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(tiles, 1, 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = (size_t)a.smem_bytes;
  lc.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  if (cudaLaunchKernelEx(&lc, k_gemm_tc<1>, tmW, tmX, a) != cudaSuccess) return CS_ERR_CUDA;
  if (cs_launch_pdl(k_tile_reduce_static, dim3(rows), dim3(128), 0, st, (const float*)tile_max,
                    (const int*)tile_idx, tiles, kStaticMaxTiles, (const int*)status, ids) != cudaSuccess)
    return CS_ERR_CUDA;
  return CS_OK;
}
