// The three projections that follow attention in a decoder layer - attention output
// (+ residual), gate/up (+ SwiGLU), down (+ residual) - as ONE launch (Sec. 3.2: the
// verification forward).  Each depends on the whole output of the one before it, so as
// separate kernels every hand-over costs a kernel boundary: epilogue, CTA exit, dependent
// launch, ring refill - about 9 us with HBM idle.  Here the grid stays resident: between two
// phases the CTAs meet at a grid barrier (a global counter), and the TMA producer of every CTA
// runs ahead of that barrier, so the weight ring is already full of the next phase's tiles when
// the barrier opens.
//
// Grid = (tiles of the residual GEMMs) x (split-K factor S), plain CTAs - no clusters: a
// cluster must find all its CTAs free inside one GPC, and with other kernels still draining the
// hardware was seen to queue the last cluster behind a GPC that never frees (its occupants wait
// at the grid barrier), so only freely placeable CTAs can be guaranteed to be co-resident.  In a
// residual phase CTA (c, r) works on output tile c, K slice r; the S partial tiles go to a
// global scratch (L2-resident, 8 KB each), a per-tile counter tells when all S are there, and
// each rank finishes a slice of the features from all S partials in rank order (deterministic).
// In the gate/up phase every CTA owns one whole tile (tile = c * S + r).
//
// Residency: the grid barrier needs all CTAs on the GPU at once.  The grid is at most two CTAs
// per SM (checked once per context by a probe launch of this very kernel), no kernel launched
// later can take SM slots before the last grid barrier has been passed (the programmatic-launch
// trigger is issued only then), and every kernel launched earlier finishes without waiting for
// this one.  Every wait - mbarrier, grid barrier, tile counter - is bounded (2 s): on expiry the
// CTA flags CS_DEV_TIMEOUT and runs on to its exit.
#include <stdlib.h>
#include <string.h>

#include "cs_common.cuh"

namespace {

constexpr int kThreads = 192;
constexpr int kTileABytes = CS_GEMM_BM * CS_GEMM_BK * 2;   // 16 KB
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
constexpr int kPhases = 3;

struct ChainPhase {
  int N, K, num_kb, kb_per_split, splits, mode, F;
  float* out;               // RESIDUAL: residual stream [rows][N] fp32
  __nv_bfloat16* act;       // SWIGLU: [rows][F] leading bf16 terms
  __nv_bfloat16* act_lo;    // SWIGLU: second bf16 terms
  NormFuse nf;
};

struct ChainArgs {
  ChainPhase ph[kPhases];
  int rows, n_tok, lo_row, stages, n_ctas;
  int probe;                // 1 = only test that the whole grid is resident at once (no GEMM work)
  unsigned* bar;            // [0..1] grid-barrier counters, [8 + i * tiles + tile] tile counters of the i-th
                            // residual phase; all zero at launch
  float* scratch;           // [tiles * S][n_tok][128] split-K partial tiles
  int* status;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u) {
      if (*abort_flag) return false;
      const unsigned long long now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) return false;
    }
  }
}
// Grid barrier, waiting side: until `target` CTAs have arrived on the counter.
__device__ __noinline__ bool grid_wait(const unsigned* counter, unsigned target, volatile int* abort_flag) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const unsigned long long now = globaltimer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) return false;
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
// K-major operand tile, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// Four consecutive floats of all S partial tiles in the scratch, summed in rank order; all
// loads (L2: the partials were written by other SMs in this launch) are issued before the first add.
__device__ __forceinline__ float4 sum_partials(const float* first, size_t rank_stride, int splits) {
  float4 v[CS_MAX_SPLITS];
#pragma unroll
  for (int q = 0; q < CS_MAX_SPLITS; ++q)
    v[q] = (q < splits) ? __ldcg(reinterpret_cast<const float4*>(first + (size_t)q * rank_stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
  float4 y = v[0];
#pragma unroll
  for (int q = 1; q < CS_MAX_SPLITS; ++q) { y.x += v[q].x; y.y += v[q].y; y.z += v[q].z; y.w += v[q].w; }
  return y;
}

// which tile and which K blocks this CTA works on in a phase
struct Work {
  int tile, split, kb0, nkb;
};
__device__ __forceinline__ Work phase_work(const ChainPhase& P, int cluster_id, int rank, int S) {
  Work w;
  const int tiles = (P.N + CS_GEMM_BM - 1) / CS_GEMM_BM;
  if (P.splits > 1) {
    w.tile = cluster_id;
    w.split = rank;
    w.kb0 = rank * P.kb_per_split;
    w.nkb = max(0, min(P.num_kb, w.kb0 + P.kb_per_split) - w.kb0);
  } else {
    w.tile = cluster_id * S + rank;
    w.split = 0;
    w.kb0 = 0;
    w.nkb = P.num_kb;
  }
  if (w.tile >= tiles) w.nkb = 0;
  return w;
}

__global__ void __launch_bounds__(kThreads, 1)
k_gemm_chain(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmX0,
             const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmX1,
             const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmX2, ChainArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);   // operand tiles need 1024-byte alignment
  const int xtile = a.n_tok * 128;                               // one activation tile (one bf16 term)
  const int stage_bytes = kTileABytes + 2 * xtile;
  const int stages = a.stages;
  float* dump = reinterpret_cast<float*>(smem + (size_t)stages * stage_bytes);   // [n_tok][128] parked tile
  float* part = dump + a.n_tok * CS_GEMM_BM;                                      // [n_tok][32] sums of squares
  float* rstd_s = part + a.n_tok * 32;                                            // [n_tok]
  uint64_t* bars = reinterpret_cast<uint64_t*>(rstd_s + a.n_tok);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * stages + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_never = reinterpret_cast<volatile int*>(tmem_slot + 2);
  const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + stages), bar_acc = smem_u32(bars + 2 * stages),
                 bar_free = smem_u32(bars + 2 * stages + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = gridDim.y, cluster_id = blockIdx.x, rank = blockIdx.y;   // (tile group, K slice)
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < a.n_tok) tmem_cols <<= 1;

  if (threadIdx.x == 128) {
    for (int s = 0; s < stages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    mbar_init(bar_acc, 1);
    mbar_init(bar_free, 128);
    *s_abort = 0;
    *s_never = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!a.probe) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW0) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX0) : "memory");
    }
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (a.probe) {
    // Residency test: every CTA checks in and waits (bounded) until all have.  It succeeds
    // exactly when the grid barrier of the real launch can succeed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (threadIdx.x == 0) {
      asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.bar) : "memory");
      if (!grid_wait(a.bar, (unsigned)a.n_ctas, s_never)) atomicOr(a.status, CS_DEV_TIMEOUT);
    }
  } else if (warp == 4) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int g = 0;          // K blocks issued so far, over all phases: slot = g % stages
      int issued = 0;     // K blocks whose loads are (partly) in flight, for the drain
      bool ok = true;
      for (int p = 0; p < kPhases && ok; ++p) {
        const ChainPhase& P = a.ph[p];
        const CUtensorMap* mW = (p == 0) ? &tmW0 : (p == 1 ? &tmW1 : &tmW2);
        const CUtensorMap* mX = (p == 0) ? &tmX0 : (p == 1 ? &tmX1 : &tmX2);
        const Work w = phase_work(P, cluster_id, rank, S);
        const int n0 = w.tile * CS_GEMM_BM;
        // weights depend on nothing: fill the ring with this phase's first tiles before its inputs exist
        const int npre = min(w.nkb, stages);
        int pre = 0;
        for (; pre < npre; ++pre) {
          const int gi = g + pre, s = gi % stages;
          if (!mbar_wait(bar_empty + 8 * s, (((uint32_t)(gi / stages)) & 1u) ^ 1u, s_abort)) { ok = false; break; }
          mbar_expect_tx(bar_full + 8 * s, (uint32_t)stage_bytes);
          tma_load_2d(smem_u32(smem + (size_t)s * stage_bytes), mW, bar_full + 8 * s, (w.kb0 + pre) * CS_GEMM_BK, n0);
          issued = gi + 1;
        }
        if (!ok) break;
        if (p == 0) {
          asm volatile("griddepcontrol.wait;" ::: "memory");
        } else if (!grid_wait(a.bar + (p - 1), (unsigned)a.n_ctas, s_abort)) {
          ok = false;
          break;
        }
        // from here on the whole grid is known to be resident: later kernels may take SM slots
        if (p == kPhases - 1) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        asm volatile("fence.proxy.async;" ::: "memory");   // peers' generic-proxy stores before the TMA reads them
        for (int i = 0; i < pre; ++i) {
          const int gi = g + i, s = gi % stages;
          const uint32_t sx = smem_u32(smem + (size_t)s * stage_bytes) + kTileABytes;
          tma_load_2d(sx, mX, bar_full + 8 * s, (w.kb0 + i) * CS_GEMM_BK, 0);
          tma_load_2d(sx + xtile, mX, bar_full + 8 * s, (w.kb0 + i) * CS_GEMM_BK, a.lo_row);
        }
        for (int i = pre; i < w.nkb; ++i) {
          const int gi = g + i, s = gi % stages;
          if (!mbar_wait(bar_empty + 8 * s, (((uint32_t)(gi / stages)) & 1u) ^ 1u, s_abort)) { ok = false; break; }
          const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
          mbar_expect_tx(bar_full + 8 * s, (uint32_t)stage_bytes);
          tma_load_2d(sa, mW, bar_full + 8 * s, (w.kb0 + i) * CS_GEMM_BK, n0);
          tma_load_2d(sa + kTileABytes, mX, bar_full + 8 * s, (w.kb0 + i) * CS_GEMM_BK, 0);
          tma_load_2d(sa + kTileABytes + xtile, mX, bar_full + 8 * s, (w.kb0 + i) * CS_GEMM_BK, a.lo_row);
          issued = gi + 1;
        }
        g += w.nkb;
      }
      if (!ok) {
        *s_abort = 1;
        atomicOr(a.status, CS_DEV_TIMEOUT);
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      }
      if (*s_abort) {
        // copies still in flight must land before this CTA's shared memory is released
        // (a block whose activation half was never issued runs into the time limit instead)
        for (int j = max(0, issued - stages); j < issued; ++j)
          mbar_wait(bar_full + 8 * (j % stages), (uint32_t)(j / stages) & 1u, s_never);
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(a.n_tok >> 3) << 17) |
                             ((uint32_t)(CS_GEMM_BM >> 4) << 24);
      int g = 0;
      bool ok = true;
      for (int p = 0; p < kPhases && ok; ++p) {
        const Work w = phase_work(a.ph[p], cluster_id, rank, S);
        // the accumulator of the previous phase has been read out
        if (p > 0 && !mbar_wait(bar_free, (uint32_t)(p - 1) & 1u, s_abort)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (int i = 0; i < w.nkb; ++i) {
          const int gi = g + i, s = gi % stages;
          if (!mbar_wait(bar_full + 8 * s, (uint32_t)(gi / stages) & 1u, s_abort)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
          const uint64_t da = umma_desc(sa), db = umma_desc(sa + kTileABytes), dl = umma_desc(sa + kTileABytes + xtile);
#pragma unroll
          for (int kk = 0; kk < CS_GEMM_BK / 16; ++kk) {
            umma_bf16(tmem_base, da + 2 * kk, db + 2 * kk, idesc, (i > 0 || kk > 0) ? 1u : 0u);
            umma_bf16(tmem_base, da + 2 * kk, dl + 2 * kk, idesc, 1u);   // x = hi + lo
          }
          umma_commit(bar_empty + 8 * s);
        }
        if (!ok) break;
        umma_commit(bar_acc);
        g += w.nkb;
      }
      if (!ok) {
        *s_abort = 1;
        atomicOr(a.status, CS_DEV_TIMEOUT);
        umma_commit(bar_acc);
      }
    }
  } else {
    // ------------------------------------------------------------- read-out, reduction, epilogues (warps 0-3)
    const int e = threadIdx.x;
    int sp = 0;                 // residual (split) phases finished so far
    bool ok = true;
    for (int p = 0; p < kPhases; ++p) {
      const ChainPhase& P = a.ph[p];
      const Work w = phase_work(P, cluster_id, rank, S);
      const int n0 = w.tile * CS_GEMM_BM;
      // what the previous phase (or the previous kernel) wrote is complete and visible
      if (p == 0) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
      } else {
        // one poller per CTA besides the producer; the named barrier hands its result on
        if (e == 0 && !grid_wait(a.bar + (p - 1), (unsigned)a.n_ctas, s_abort)) *s_abort = 1;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        ok = (*s_abort == 0);
      }
      const bool scaled = P.nf.ssq_in != nullptr;
      if (ok && scaled) {
        for (int tok = warp; tok < a.rows; tok += 4) {
          float ss = 0.f;
          for (int sl = lane; sl < P.nf.slots_in; sl += 32) ss += __ldcg(P.nf.ssq_in + (size_t)tok * P.nf.slot_stride + sl);   // written by other SMs in this launch: L2, not L1
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
          if (lane == 0) rstd_s[tok] = rsqrtf(ss * P.nf.inv_d + P.nf.eps);
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (ok) ok = mbar_wait(bar_acc, (uint32_t)p & 1u, s_abort);
      ok = __all_sync(0xffffffffu, ok) && (*s_abort == 0);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (!ok) {
        if (lane == 0) { *s_abort = 1; atomicOr(a.status, CS_DEV_TIMEOUT); }
        break;
      }
      for (int c0 = 0; c0 < a.n_tok && c0 < a.rows; c0 += 16) {
        uint32_t v[16];
        if (w.nkb > 0) {
          tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0u;
        }
        float* park = (P.splits > 1) ? a.scratch + ((size_t)(w.tile * P.splits + w.split) * a.n_tok) * CS_GEMM_BM : dump;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          float f = __uint_as_float(v[j]);
          if (scaled && c0 + j < a.rows) f *= rstd_s[c0 + j];
          park[(c0 + j) * CS_GEMM_BM + warp * 32 + lane] = f;
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(bar_free);
      asm volatile("bar.sync 1, 128;" ::: "memory");   // tile parked
      const bool split_phase = P.splits > 1;
      if (split_phase) {
        // all S partial tiles of this output tile are in the scratch
        unsigned* cnt = a.bar + 8 + sp * gridDim.x + w.tile;
        if (e == 0) {
          __threadfence();
          asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(cnt) : "memory");
          if (!grid_wait(cnt, (unsigned)P.splits, s_abort)) *s_abort = 1;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        ok = (*s_abort == 0);
      }
      if (P.mode == CS_EPI_SWIGLU) {
        // features 0..63 of the tile are gate rows, 64..127 the matching up rows
        const int total = 16 * a.rows;
        if (w.nkb > 0)
          for (int idx = e; idx < total; idx += 128) {
            const int j = 4 * (idx & 15), tok = idx >> 4;
            const float4 g4 = *reinterpret_cast<const float4*>(dump + tok * CS_GEMM_BM + j);
            const float4 u4 = *reinterpret_cast<const float4*>(dump + tok * CS_GEMM_BM + 64 + j);
            const float gv[4] = {g4.x, g4.y, g4.z, g4.w}, uv[4] = {u4.x, u4.y, u4.z, u4.w};
            const int jj0 = w.tile * 64 + j;
            if (jj0 + 3 < P.F) {
              float v4[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) v4[i] = gv[i] / (1.f + expf(-gv[i])) * uv[i];
              __nv_bfloat162 h[2], l[2];
              h[0] = __floats2bfloat162_rn(v4[0], v4[1]); h[1] = __floats2bfloat162_rn(v4[2], v4[3]);
              const float2 h0 = __bfloat1622float2(h[0]), h1 = __bfloat1622float2(h[1]);
              l[0] = __floats2bfloat162_rn(v4[0] - h0.x, v4[1] - h0.y); l[1] = __floats2bfloat162_rn(v4[2] - h1.x, v4[3] - h1.y);
              *reinterpret_cast<uint2*>(P.act + (size_t)tok * P.F + jj0) = *reinterpret_cast<const uint2*>(h);
              *reinterpret_cast<uint2*>(P.act_lo + (size_t)tok * P.F + jj0) = *reinterpret_cast<const uint2*>(l);
            }
          }
      } else {
        // residual update: each rank finishes a slice of the tile's features, four per thread
        const int fs = ((CS_GEMM_BM + P.splits - 1) / P.splits + 3) & ~3;
        const int f_lo = w.split * fs, f_n = max(0, min(CS_GEMM_BM, f_lo + fs) - f_lo);
        const int per_tok = f_n >> 2;
        const bool feeds_norm = P.nf.gain_out != nullptr;
        const int total = ok ? per_tok * a.rows : 0;
        for (int idx = e; idx < total; idx += 128) {
          const int f = f_lo + 4 * (idx % per_tok), tok = idx / per_tok;
          float4 y;
          if (split_phase)
            y = sum_partials(a.scratch + ((size_t)(w.tile * P.splits) * a.n_tok + tok) * CS_GEMM_BM + f,
                             (size_t)a.n_tok * CS_GEMM_BM, P.splits);
          else y = *reinterpret_cast<const float4*>(dump + tok * CS_GEMM_BM + f);
          float ssq = 0.f;
          if (n0 + f + 3 < P.N) {
            float* dst = P.out + (size_t)tok * P.N + n0 + f;
            const float4 x = __ldcg(reinterpret_cast<const float4*>(dst));
            const float4 o = make_float4(x.x + y.x, x.y + y.y, x.z + y.z, x.w + y.w);
            *reinterpret_cast<float4*>(dst) = o;
            if (feeds_norm) {
              const uint2 gw = *reinterpret_cast<const uint2*>(P.nf.gain_out + n0 + f);
              const float2 g01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw.x));
              const float2 g23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw.y));
              const float w0 = o.x * g01.x, w1 = o.y * g01.y, w2 = o.z * g23.x, w3 = o.w * g23.y;
              __nv_bfloat162 h[2], l[2];
              h[0] = __floats2bfloat162_rn(w0, w1); h[1] = __floats2bfloat162_rn(w2, w3);
              const float2 h0 = __bfloat1622float2(h[0]), h1 = __bfloat1622float2(h[1]);
              l[0] = __floats2bfloat162_rn(w0 - h0.x, w1 - h0.y); l[1] = __floats2bfloat162_rn(w2 - h1.x, w3 - h1.y);
              __nv_bfloat16* xo = P.nf.xn_out + (size_t)tok * P.N + n0 + f;
              *reinterpret_cast<uint2*>(xo) = *reinterpret_cast<const uint2*>(h);
              *reinterpret_cast<uint2*>(xo + (size_t)CS_MAX_ROWS * P.N) = *reinterpret_cast<const uint2*>(l);
              ssq = (o.x * o.x + o.y * o.y) + (o.z * o.z + o.w * o.w);
            }
          }
          if (feeds_norm) part[tok * 32 + idx % per_tok] = ssq;
        }
        if (feeds_norm) {
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (ok)
            for (int tok = e; tok < a.rows; tok += 128) {
              float ss = 0.f;
              for (int q = 0; q < per_tok; ++q) ss += part[tok * 32 + q];
              P.nf.ssq_out[(size_t)tok * P.nf.slot_stride + w.tile * P.splits + w.split] = ss;
            }
        }
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");   // partials read, global stores issued
      if (split_phase) ++sp;
      if (p < kPhases - 1 && e == 0) {
        __threadfence();
        asm volatile("fence.proxy.async;" ::: "memory");
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.bar + p) : "memory");
      }
      if (!ok) {
        if (lane == 0) { *s_abort = 1; atomicOr(a.status, CS_DEV_TIMEOUT); }
        break;
      }
    }
  }
  // ---------------------------------------------------------------- teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 5) {
    if (*s_abort && lane == 0) mbar_wait(bar_acc, (uint32_t)(kPhases - 1) & 1u, s_never);   // MMAs retired (bounded)
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

}  // namespace

// Attention-output, gate/up and down projections of one layer in one launch.  Returns
// CS_ERR_UNSUPPORTED (nothing launched, ctx->err untouched) when the layer's plans or the
// block height do not fit the chain's grid; the caller then launches the three GEMMs one by one.
cs_status cs_launch_gemm_chain(cs_ctx* ctx, const LayerPlan* L, int rows, const NormFuse* nf_o, const NormFuse* nf_gate_up,
                               const NormFuse* nf_down, cudaStream_t st) {
  const cs_model_config& c = ctx->cfg;
  const GemmPlan* g[kPhases] = {&L->o, &L->gate_up, &L->down};
  const int S = L->o.splits, T = cs_ceil_div(L->o.N, CS_GEMM_BM);
  if (ctx->chain_state <= 0 || S < 2 || L->down.splits != S || L->gate_up.splits != 1 || L->down.N != L->o.N ||
      cs_ceil_div(L->gate_up.N, CS_GEMM_BM) > T * S || (c.d_ffn & 3) != 0 || (L->o.N & 3) != 0 || T * S > 2 * ctx->num_sms || 8 + 2 * T > CS_CHAIN_BAR_WORDS) {
    return CS_ERR_UNSUPPORTED;
  }
  ChainArgs a;
  a.rows = rows;
  a.n_tok = cs_ceil_div(rows, 16) * 16;
  a.lo_row = CS_MAX_ROWS;
  a.n_ctas = T * S;
  a.probe = 0;
  a.bar = ctx->chain_bar;
  a.scratch = ctx->chain_scratch;
  a.status = ctx->d_status;
  if (a.n_tok > CS_CHAIN_MAX_TOK) return CS_ERR_UNSUPPORTED;
  const int stage_bytes = kTileABytes + 2 * a.n_tok * 128;
  const int fixed = 1024 + a.n_tok * (CS_GEMM_BM + 32 + 1) * 4 + (2 * 8 + 4) * 8 + 16;
  int stages = (113 * 1024 - fixed) / stage_bytes;      // two CTAs per SM
  if (stages > 8) stages = 8;
  if (stages < 4) return CS_ERR_UNSUPPORTED;
  a.stages = stages;
  const size_t smem = (size_t)fixed + (size_t)stages * stage_bytes;
  const NormFuse* nf[kPhases] = {nf_o, nf_gate_up, nf_down};
  const int modes[kPhases] = {CS_EPI_RESIDUAL, CS_EPI_SWIGLU, CS_EPI_RESIDUAL};
  for (int p = 0; p < kPhases; ++p) {
    ChainPhase& P = a.ph[p];
    P.N = g[p]->N;
    P.K = g[p]->K;
    P.num_kb = cs_ceil_div(g[p]->K, CS_GEMM_BK);
    P.kb_per_split = g[p]->kb_per_split;
    P.splits = g[p]->splits;
    P.mode = modes[p];
    P.F = c.d_ffn;
    P.out = ctx->x;
    P.act = ctx->act;
    P.act_lo = ctx->act + (size_t)CS_MAX_ROWS * c.d_ffn;
    P.nf = NormFuse{};
    if (nf[p] != nullptr) P.nf = *nf[p];
  }
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(T, S, 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  lc.numAttrs = 1;
  CS_CUDA_OK(ctx, cudaLaunchKernelEx(&lc, k_gemm_chain, L->o.tmW, ctx->tmAttn, L->gate_up.tmW, ctx->tmXn, L->down.tmW,
                                     ctx->tmAct, a));
  return CS_OK;
}

// Decide once, when the context is created, whether this GPU holds the chain's whole grid at
// once (two CTAs per SM).  The occupancy calculator
// under-reports kernels that allocate tensor memory, so the question is put to the hardware:
// the same kernel, with the same launch shape and shared-memory footprint as a decode-sized
// launch, only checks in at the grid barrier.  Synchronises the stream; not for use during capture.
void cs_gemm_chain_probe(cs_ctx* ctx, cudaStream_t st) {
  if (ctx->chain_state != 0) return;
  ctx->chain_state = -1;
  const LayerPlan* L = &ctx->layers[0];
  const int S = L->o.splits, T = cs_ceil_div(L->o.N, CS_GEMM_BM);
  if (S < 2 || L->down.splits != S || L->gate_up.splits != 1 || T * S > 2 * ctx->num_sms) return;
  ChainArgs a;
  memset(&a, 0, sizeof(a));
  a.n_tok = 16;
  a.n_ctas = T * S;
  a.probe = 1;
  a.bar = ctx->chain_bar;
  a.status = ctx->d_status;
  const int stage_bytes = kTileABytes + 2 * a.n_tok * 128;
  const int fixed = 1024 + a.n_tok * (CS_GEMM_BM + 32 + 1) * 4 + (2 * 8 + 4) * 8 + 16;
  int stages = (113 * 1024 - fixed) / stage_bytes;
  if (stages > 8) stages = 8;
  a.stages = stages;
  if (cudaFuncSetAttribute(k_gemm_chain, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024) != cudaSuccess) {
    cudaGetLastError();
    return;
  }
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(T, S, 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = (size_t)fixed + (size_t)stages * stage_bytes;
  lc.stream = st;
  lc.attrs = nullptr;
  lc.numAttrs = 0;
  int bits = -1;
  if (cudaMemsetAsync(ctx->chain_bar, 0, CS_CHAIN_BAR_WORDS * sizeof(unsigned), st) != cudaSuccess ||
      cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st) != cudaSuccess ||
      cudaLaunchKernelEx(&lc, k_gemm_chain, L->o.tmW, L->o.tmW, L->o.tmW, L->o.tmW, L->o.tmW, L->o.tmW, a) != cudaSuccess ||
      cudaMemcpyAsync(&bits, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return;
  }
  if (bits == 0) ctx->chain_state = 1;
}
