// Causal block attention over the bf16 KV cache on the 5th-generation tensor cores
// (Sec. 3.2; App. B.2), for head_dim 128.
//
// One CTA = one (sequence, KV head), one slice of the key range and one group of block rows (the
// (k+1) block rows of the G query heads sharing the KV head: at most 96 query rows per group).
// The cached keys and the head dims are the M dimension of the two products and the query rows
// the N dimension, so the operand traffic scales with the real number of query rows (44 for an
// 11-row block of a 4:1 GQA model) instead of a padded 128:
//     S^T [128 keys x NQ]  = K_tile Q_hi^T + K_tile Q_lo^T     (A = K tile, K-major; B = Q, K-major)
//     O^T [128 dims x NQ]  = V_tile^T P_hi^T + V_tile^T P_lo^T (A = V tile, MN-major straight from the
//                                                               cache layout; B = P^T, MN-major)
// Queries and softmax weights enter as two bf16 terms each, so they are fp32-equivalent and only
// K and V - which the cache stores in bf16 - are rounded.  A tcgen05.mma of these shapes keeps
// its issuer busy for about 114 cycles whatever N is (measured for N from 32 to 192), so the
// two terms of the second operand are laid side by side along N - [Q_hi; Q_lo] as one operand of
// 2 NQ rows, [P_hi^T | P_lo^T] as one of 2 NQ columns - and one instruction per 16 K-elements
// does the work of two; the two halves of the accumulator are added where it is read (S^T keeps
// one NQ-wide accumulator and two instructions when TMEM has no room for 2 NQ columns twice).
// TMEM lane = key (S^T) or head dim (O^T), column = query row.  Softmax: twelve warps in three
// column groups; thread t of a lane quarter owns key t of the tile and a third of the query
// columns (warps w, w + 4 and w + 8 share the lanes).  Each column has a running reference point
// m for its exponentials, which follows the column's true maximum only from afar: it moves when
// a score exceeds it by more than 2^8.  Softmax does not depend on the reference point, and
// weights up to 2^8 are as exact in two bf16 terms as weights up to 1.  So on most tiles a
// thread only compares its scores with the columns' thresholds and the threads of a column
// group vote (one predicate-reducing barrier); the true maxima (a butterfly of 31 shuffles per
// warp plus a four-entry combine through shared memory), the correction of the sums and the
// rescaling of O^T in TMEM happen only on the few tiles where a reference point moves.  The
// weights pass works on column pairs with the packed fp32 instructions (fma / add / sub .f32x2).
// Each thread keeps its own share of every column's sum;
// the shares are added up once at the end.  P^T is written as one swizzled 16-byte chunk per 8
// columns into the row of the thread's key, which is exactly the MN-major operand layout, so
// nothing is transposed.  S^T is double-buffered in TMEM: the score product of tile i+1 runs
// during the softmax of tile i.  Blocks of up to 48 query rows have room for four S^T buffers:
// their softmax takes the key tiles two at a time (one wait, one vote, two sets of weights).
// K tiles move through a two-stage TMA ring and V tiles through a one- or two-stage ring, each
// fed by its own producer thread, so K runs a tile ahead.  Each CTA
// writes its un-normalised (O, m, sum); k_attn_merge combines the key slices.  When the caller
// vouches for the cached lengths (kv_len_early), tiles that lie wholly below the cached length
// are requested before the wait for the preceding kernel: those rows were written by earlier
// steps.  Every wait is bounded (2 s by default): on expiry the CTA flags CS_DEV_TIMEOUT, drains
// its copies, frees its TMEM and returns; the decision to give up is made uniform across the
// softmax threads by a predicate-reducing barrier, so no thread is left behind at a barrier.
#include <stdlib.h>

#include "cs_common.cuh"

namespace {

constexpr int kSoftWarps = 12, kSoftThreads = kSoftWarps * 32;   // three column groups of four warps (one per TMEM lane quarter)
constexpr int kThreads = 480;   // warps 0-11 softmax/epilogue, warp 12 K/Q producer, warp 13 MMA, warp 14 V producer
constexpr int kProdWarp = 12, kMmaWarp = 13, kVProdWarp = 14;   // (a warp of its own each: a lane that sleeps in a
                                                              //  barrier wait would hold up the other lanes of its warp)
constexpr int kTileKeys = 128;
constexpr int kDh = 128;
constexpr int kHalfBytes = kTileKeys * 128;          // one [128 keys x 64 dims] half tile (also one P^T atom)
constexpr int kNQMax = 96;                           // query rows per CTA
constexpr int kCols = kNQMax / 3;                    // query columns per softmax thread, at most
constexpr int kCtlBytes = 192;                       // 16 mbarriers + TMEM slot + flags

struct AttnArgs {
  const int* row_lim;
  const int* kv_len_early;   // cached lengths that no kernel in flight changes, or NULL
  int layer, R, Rg, G, H, Hkv, max_batch, max_seq, nsplit, NQ, rows, vstages, pbufs, qstack;   // Rg = block rows per row group; pbufs = P^T buffers (1 or 2)
  int smem_bytes;            // dynamic shared memory of the launch
  float scale_log2e;
  float* out_o;
  float* out_ml;
  int* status;
  unsigned long long wait_ns;   // limit of every bounded wait
  unsigned long long* stamp;    // step timeline slot of this launch, or NULL
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
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// operand descriptors, 128-byte swizzle.  K-major: rows of 128 bytes, 8-row groups 1024 bytes
// apart.  MN-major: rows (one per K index) of 128 bytes holding 64 contiguous MN elements,
// 8-row groups 1024 bytes apart (stride field), the next 64 MN elements `lbo` bytes further.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr, uint32_t lbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
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
// eight accumulator columns of this thread's lane (no wait: several loads share one wait)
__device__ __forceinline__ void tmem_ld8_nowait(uint32_t taddr, float* v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// The loaded registers are only valid after the wait, which the compiler cannot know: this empty
// statement, placed behind the wait, redefines them, so no use of theirs is scheduled ahead of it.
__device__ __forceinline__ void tmem_landed8(float* v) {
  asm volatile("" : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7])::"memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const float* v) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
                 "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
                 "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7]))
               : "memory");
}
// 2^x, hardware approximation (relative error about 2^-22; -inf gives 0)
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Two fp32 values in one 64-bit register and the packed fp32 arithmetic of this architecture
// (fma / add / sub on both halves in one instruction): the weights pass works on column pairs.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 r, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
  f32x2 d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// Maximum over the 32 lanes of each of 32 per-lane values with 31 shuffles (instead of five per
// value): every step halves the values a lane is responsible for - it keeps one half of its array,
// combined with what its partner sends of the same half - so that lane L ends up with the
// maximum of x[L] over the warp.
__device__ __forceinline__ float warp_max32(float (&x)[32], int lane) {
#pragma unroll
  for (int w = 16; w >= 1; w >>= 1) {
    const bool up = (lane & w) != 0;
#pragma unroll
    for (int j = 0; j < w; ++j) {
      const float send = up ? x[j] : x[j + w];
      const float keep = up ? x[j + w] : x[j];
      x[j] = fmaxf(keep, __shfl_xor_sync(0xffffffffu, send, w));
    }
  }
  return x[0];
}
// barrier of one column group of the softmax threads (128 threads, ids 1 to 3) that also ANDs a predicate:
// every thread learns whether all of them are still fine, so they leave their loops together
__device__ __forceinline__ bool group_all(int id, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n.reg .pred p, q;\nsetp.ne.b32 p, %2, 0;\nbar.red.and.pred q, %1, 128, p;\nselp.u32 %0, 1, 0, q;\n}"
      : "=r"(out) : "r"(id), "r"((uint32_t)pred) : "memory");
  return out != 0;
}
// the same barrier with OR: does any thread of the group raise the predicate?
__device__ __forceinline__ bool group_any(int id, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n.reg .pred p, q;\nsetp.ne.b32 p, %2, 0;\nbar.red.or.pred q, %1, 128, p;\nselp.u32 %0, 1, 0, q;\n}"
      : "=r"(out) : "r"(id), "r"((uint32_t)pred) : "memory");
  return out != 0;
}

// KC = query columns per softmax thread at most (register arrays), NSB = S^T buffers in TMEM: 2, or 4
// for blocks of up to 48 query rows, whose softmax then takes the key tiles two at a time.
template <int KC, int NSB>
__global__ void __launch_bounds__(kThreads, 1)
k_attn_tcw(const __grid_constant__ CUtensorMap tmKV, const __grid_constant__ CUtensorMap tmQ, AttnArgs a) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  // blockIdx.z picks a group of Rg consecutive block rows (blocks taller than 96 / G rows)
  const int NQ = a.NQ, G = a.G, R = a.R, r0 = blockIdx.z * a.Rg, Rcur = min(a.Rg, R - r0);
  const int nq = G * Rcur, nq_box = G * a.Rg, vstages = a.vstages;
  const int natoms = (2 * NQ + 63) >> 6;               // 64-column atoms of P^T (both terms side by side)
  const uint32_t qhalf = (uint32_t)NQ * 128u;          // [NQ rows x 64 dims] of one term
  const uint32_t pbuf = (uint32_t)natoms * kHalfBytes; // [atom][128 keys][128 B]
  uint8_t* sQ = smem;                                  // [half][term][NQ][128 B]: per dim half, the 2 NQ rows of both terms in a row
  uint8_t* sP = sQ + 4 * qhalf;                        // [buffer][atom][128 keys][128 B]: columns q (leading terms) and NQ + q
  uint8_t* sK = sP + (size_t)a.pbufs * pbuf;                        // [2 stages][half][128 keys][128 B]
  uint8_t* sV = sK + 2 * 2 * kHalfBytes;               // [vstages][half][128 keys][128 B]
  uint8_t* ctl = sV + (size_t)vstages * 2 * kHalfBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ctl);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 20);
  volatile int* s_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_never = reinterpret_cast<volatile int*>(tmem_slot + 2);
  int* s_lmax = reinterpret_cast<int*>(tmem_slot + 3);
  int* s_limmin = reinterpret_cast<int*>(tmem_slot + 4);     // fewest keys any live query row of the group attends to
  int* s_lim = reinterpret_cast<int*>(ctl + kCtlBytes);                 // [NQ] keys each query row attends to
  float* s_priv = reinterpret_cast<float*>(s_lim + kNQMax);             // [12 warps][3][kCols] each warp's copy of its columns' reference points
  float* s_red = reinterpret_cast<float*>(s_priv + kSoftWarps * 3 * kCols);   // [2][12 warps][kCols] per-warp column maxima / sums, by tile parity
  if ((size_t)(reinterpret_cast<uint8_t*>(s_red + 2 * kSoftWarps * kCols) - smem_raw) > (size_t)a.smem_bytes) {
    if (threadIdx.x == 0) atomicOr(a.status, CS_DEV_SMEM);   // the launcher sizes the window for exactly this layout
    return;
  }
  const uint32_t b_kfull = smem_u32(bars), b_kfree = smem_u32(bars + 2), b_vfull = smem_u32(bars + 4),
                 b_vfree = smem_u32(bars + 6), b_qfull = smem_u32(bars + 8), b_sready = smem_u32(bars + 16),   // b_sready: one per S^T buffer (bars 16-19)
                 b_pready = smem_u32(bars + 14), b_odone = smem_u32(bars + 12);   // b_pready (bars 14, 15) and b_odone: two barriers each, by tile parity

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.x / a.Hkv, kvh = blockIdx.x % a.Hkv, split = blockIdx.y;
  // TMEM columns: S^T of even tiles, S^T of odd tiles (each NQ wide, or 2 NQ when the two query terms
  // are kept apart), then O^T, 2 NQ wide: the leading and the trailing weight terms' shares
  const uint32_t cstride = (uint32_t)(((a.qstack ? 2 * NQ : NQ) + 31) & ~31);
  const uint32_t ocol = NSB * cstride;
  uint32_t tmem_cols = 32;
  while (tmem_cols < ocol + (uint32_t)((2 * NQ + 31) & ~31)) tmem_cols <<= 1;

  if (tid == kProdWarp * 32) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(b_kfull + 8 * s, 1); mbar_init(b_kfree + 8 * s, 1);
      mbar_init(b_vfull + 8 * s, 1); mbar_init(b_vfree + 8 * s, 1);
    }
    for (int s = 0; s < NSB; ++s) mbar_init(b_sready + 8 * s, 1);
    mbar_init(b_qfull, 1);
    mbar_init(b_pready, kSoftThreads); mbar_init(b_pready + 8, kSoftThreads);
    mbar_init(b_odone, 1); mbar_init(b_odone + 8, 1);
    *s_abort = 0; *s_never = 0; *s_lmax = 0; *s_limmin = 0x7fffffff;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmKV) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmQ) : "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  // Slice `split` works on key tiles split, split + nsplit, ...  Its first tiles are known before
  // the key range is, so they are requested while the range is worked out (a slice beyond the
  // range only has to let them land).
  const long long krow = ((((long long)a.layer * 2 + 0) * a.max_batch + b) * a.Hkv + kvh) * (long long)a.max_seq;
  const long long vrow = ((((long long)a.layer * 2 + 1) * a.max_batch + b) * a.Hkv + kvh) * (long long)a.max_seq;
  auto load_k = [&](int i) {
    const int s = i & 1, key0 = (split + i * a.nsplit) * kTileKeys;
    const uint32_t dk = smem_u32(sK + (size_t)s * 2 * kHalfBytes);
    mbar_expect_tx(b_kfull + 8 * s, 2u * kHalfBytes);
    tma_load_2d(dk, &tmKV, b_kfull + 8 * s, 0, (int)(krow + key0));
    tma_load_2d(dk + kHalfBytes, &tmKV, b_kfull + 8 * s, 64, (int)(krow + key0));
  };
  auto load_v = [&](int i) {
    const int s = i % vstages, key0 = (split + i * a.nsplit) * kTileKeys;
    const uint32_t dv = smem_u32(sV + (size_t)s * 2 * kHalfBytes);
    mbar_expect_tx(b_vfull + 8 * s, 2u * kHalfBytes);
    tma_load_2d(dv, &tmKV, b_vfull + 8 * s, 0, (int)(vrow + key0));
    tma_load_2d(dv + kHalfBytes, &tmKV, b_vfull + 8 * s, 64, (int)(vrow + key0));
  };
  // tiles of cached keys only: nothing in flight writes them, so they need not wait for the
  // preceding kernel.  n_early = tiles of this slice this producer lane requested before the wait.
  int n_early = 0;
  if ((warp == kProdWarp || warp == kVProdWarp) && lane == 0 && a.kv_len_early != nullptr) {
    const int cached = min(a.kv_len_early[b], a.max_seq);
    const int want = (warp == kProdWarp) ? 2 : vstages;
    while (n_early < want && (split + n_early * a.nsplit + 1) * kTileKeys <= cached) {
      if (warp == kProdWarp) load_k(n_early); else load_v(n_early);
      ++n_early;
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp < kSoftWarps) {
    int lm = 0, ln = 0x7fffffff;
    for (int r = tid; r < Rcur; r += kSoftThreads) {
      const int v = a.row_lim[b * R + r0 + r];
      lm = max(lm, v);
      ln = min(ln, v);
    }
    lm = __reduce_max_sync(0xffffffffu, lm);
    ln = __reduce_min_sync(0xffffffffu, ln);
    if (lane == 0 && lm > 0) atomicMax(s_lmax, lm);
    if (lane == 0) atomicMin(s_limmin, ln);
    for (int q = tid; q < NQ; q += kSoftThreads) {
      s_lim[q] = (q < nq) ? a.row_lim[b * R + r0 + q / G] : 0;
    }
  }
  if (warp == kProdWarp && lane == 0) {
    // tile 0 of K first (the first product waits for it), then the queries (fresh in L2)
    if (n_early < 1) load_k(0);
    mbar_expect_tx(b_qfull, (uint32_t)(4 * nq_box * 128));
    for (int term = 0; term < 2; ++term)
      for (int dh = 0; dh < 2; ++dh)
        tma_load_3d(smem_u32(sQ + (2 * dh + term) * qhalf), &tmQ, b_qfull, dh * 64, kvh * G,
                    term * CS_MAX_ROWS + b * R + r0);   // the box is always Rg rows tall; rows past the group are never used
  }
  if (warp == kVProdWarp && lane == 0 && n_early < 1) load_v(0);
  __syncthreads();
  const int lmax = *s_lmax;
  const int ntiles = (lmax + kTileKeys - 1) / kTileKeys;
  const int ntl = (ntiles > split) ? (ntiles - split + a.nsplit - 1) / a.nsplit : 0;

  if (warp == kProdWarp || warp == kVProdWarp) {
    // ------------------------------------------------------------------ TMA producers: one warp feeds K, one feeds V
    if (lane == 0) {
      const bool is_k = warp == kProdWarp;
      const int st = is_k ? 2 : vstages;
      const uint32_t bfree = is_k ? b_kfree : b_vfree, bfull = is_k ? b_kfull : b_vfull;
      int issued = max(1, n_early);                     // tiles requested so far (tile 0 always is)
      bool ok = true;
      for (int i = issued; i < ntl; ++i) {
        const int s = i % st;
        if (i >= st && !mbar_wait(bfree + 8 * s, (uint32_t)(i / st - 1) & 1u, s_abort, a.wait_ns)) { ok = false; break; }
        if (is_k) load_k(i); else load_v(i);
        issued = i + 1;
      }
      if (!ok) { *s_abort = 1; atomicOr(a.status, CS_DEV_TIMEOUT); }
      // copies that nobody will consume (the CTA gave up, or tiles requested early beyond the key
      // range) must land before the shared memory goes away
      if (*s_abort || issued > ntl) {
        if (is_k) mbar_wait(b_qfull, 0, s_never, a.wait_ns);
        for (int j = max(0, issued - st); j < issued; ++j) mbar_wait(bfull + 8 * (j % st), (uint32_t)(j / st) & 1u, s_never, a.wait_ns);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && ntl > 0) {
      // bf16 x bf16 -> fp32, M = 128.  An instruction costs about the same for any N up to 200, so
      // the two bf16 terms of the second operand sit side by side along N wherever TMEM has the
      // columns: one instruction then does the work of two, and the two halves of the result are
      // added when they are read.
      auto idesc = [](int n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24); };
      const uint32_t idesc_s = idesc(a.qstack ? 2 * NQ : NQ);
      const uint32_t idesc_o = idesc(2 * NQ) | (1u << 15) | (1u << 16);   // A (= V) and B (= P^T) are MN-major
      const uint32_t aq = smem_u32(sQ), ap = smem_u32(sP);
      auto issue_scores = [&](int i) -> bool {
        const int s = i & 1, sb = i & (NSB - 1);           // K stage, S^T buffer
        if (!mbar_wait(b_kfull + 8 * s, (uint32_t)(i >> 1) & 1u, s_abort, a.wait_ns)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t ak = smem_u32(sK + (size_t)s * 2 * kHalfBytes);
        const uint32_t acc = tmem_base + (uint32_t)sb * cstride;
        if (a.qstack) {
#pragma unroll
          for (int dh = 0; dh < 2; ++dh)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_bf16(acc, desc_kmajor(ak + dh * kHalfBytes) + 2 * kk, desc_kmajor(aq + dh * 2 * qhalf) + 2 * kk, idesc_s,
                        (dh | kk) ? 1u : 0u);
        } else {
#pragma unroll
          for (int term = 0; term < 2; ++term)
#pragma unroll
            for (int dh = 0; dh < 2; ++dh)
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                umma_bf16(acc, desc_kmajor(ak + dh * kHalfBytes) + 2 * kk, desc_kmajor(aq + (2 * dh + term) * qhalf) + 2 * kk,
                          idesc_s, (term | dh | kk) ? 1u : 0u);
        }
        umma_commit(b_kfree + 8 * s);
        umma_commit(b_sready + 8 * sb);
        return true;
      };
      bool ok = mbar_wait(b_qfull, 0, s_abort, a.wait_ns);
      int qk = 0;                                          // score products issued so far
      for (int i = 0; i < ntl && ok; ++i) {
        // The scores of the next tiles go first: they run during this tile's softmax.  The S^T buffer
        // of tile t was last read by the softmax of tile t - NSB, which had finished before P^T of
        // that tile was signalled - and this thread has waited for the P^T of every tile before i.
        // A column group whose tiles are quick - all its rows masked - can therefore be a tile ahead
        // of the others, which is why "P^T written" has a barrier per tile parity: it cannot be two
        // ahead, because the scores of tile i + 2 are only issued after P^T of tile i (with four
        // buffers the softmax hands tiles over in pairs, odd after even, so parity still tells them apart).
        while (qk < ntl && qk < i + NSB && ok) { ok = issue_scores(qk); ++qk; }
        if (!ok) break;
        const int s = i % vstages;
        if (!mbar_wait(b_pready + 8 * (i & 1), (uint32_t)(i >> 1) & 1u, s_abort, a.wait_ns) ||
            !mbar_wait(b_vfull + 8 * s, (uint32_t)(i / vstages) & 1u, s_abort, a.wait_ns)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t av = smem_u32(sV + (size_t)s * 2 * kHalfBytes);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)   // 16 keys per instruction
          umma_bf16(tmem_base + ocol, desc_mnmajor(av + kk * 2048, kHalfBytes),
                    desc_mnmajor(ap + (uint32_t)(i % a.pbufs) * pbuf + kk * 2048, kHalfBytes), idesc_o, (i > 0 || kk > 0) ? 1u : 0u);
        umma_commit(b_vfree + 8 * s);
        umma_commit(b_odone + 8 * (i & 1));
      }
      if (!ok) { *s_abort = 1; atomicOr(a.status, CS_DEV_TIMEOUT); }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    // thread = one TMEM lane (a key of the tile for S^T, a head dim for O^T) and half of the columns
    const int wq = warp & 3, grp = warp >> 2;
    const int row = wq * 32 + lane;                    // TMEM lane of this thread
    const int ncol = NQ / 3, nch = ncol >> 3;          // this thread's columns (8, 16, 24 or 32), in chunks of 8
    const int q0 = grp * ncol;
    const uint32_t lane_base = tmem_base + ((uint32_t)(wq * 32) << 16);
    const float sc = a.scale_log2e;
    f32x2 lsum[KC / 2];                             // this key lane's share of every column's sum, two columns per register pair
#pragma unroll
    for (int j = 0; j < KC / 2; ++j) lsum[j] = pack2(0.f, 0.f);
    const f32x2 sc2 = pack2(sc, sc);
    // This warp's own copy of its columns' running reference points (every warp of the group works
    // out the same values): the reference m (log2 domain), the raw score above which it has to
    // move, (m + 8) / scale, and -m for the exponent.  A column that has seen no key yet holds
    // (-inf, -inf, -inf): any finite score moves it, and a masked score gets weight 2^-inf = 0.
    // Padding columns never move (+inf) and always weigh 0.
    float* w_mo = s_priv + warp * 3 * kCols;
    float* w_thr = w_mo + kCols;
    float* w_nme = w_thr + kCols;
    for (int j = lane; j < kCols; j += 32) {
      w_mo[j] = -INFINITY;
      w_thr[j] = (q0 + j < nq) ? -INFINITY : INFINITY;
      w_nme[j] = -INFINITY;
    }
    __syncwarp();
    bool have = ntl > 0;
    const int limmin = *s_limmin;
    // ---- the pieces of one tile's softmax
    // this key's scores of this thread's columns (masked keys count as -inf)
    auto load_scores = [&](int t, float (&v)[KC]) -> bool {
      const int sb = t & (NSB - 1);
      const int tile0 = (split + t * a.nsplit) * kTileKeys;
      const bool ok = mbar_wait(b_sready + 8 * sb, (uint32_t)(t / NSB) & 1u, s_abort, a.wait_ns);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t s_addr = lane_base + (uint32_t)sb * cstride + (uint32_t)q0;
#pragma unroll
      for (int c = 0; c < KC / 8; ++c)
        if (c < nch) tmem_ld8_nowait(s_addr + 8 * c, v + 8 * c);
      if (a.qstack) {                                    // the trailing query terms' share, NQ columns further
#pragma unroll
        for (int c = 0; c < KC / 8; ++c)
          if (c < nch) {
            float w[8];
            tmem_ld8_nowait(s_addr + (uint32_t)NQ + 8 * c, w);
            tmem_ld_wait();
            tmem_landed8(w);
            tmem_landed8(v + 8 * c);                     // (requested before w: landed as well)
#pragma unroll
            for (int j = 0; j < 8; ++j) v[8 * c + j] += w[j];
          }
      } else {
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < KC / 8; ++c)
          if (c < nch) tmem_landed8(v + 8 * c);
      }
      if (tile0 + kTileKeys > limmin) {                  // some live query row masks a key of this tile
        const int key = tile0 + row;                     // the key of this lane
#pragma unroll
        for (int c = 0; c < KC / 8; ++c)
          if (c < nch) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (key >= s_lim[q0 + 8 * c + j]) v[8 * c + j] = -INFINITY;
          }
      }
      return ok;
    };
    // Does any score lie more than 2^8 above its column's reference point (or meet a column that has
    // none)?  Softmax does not depend on the reference point, and weights up to 2^8 are as exact in
    // two bf16 terms as weights up to 1, so the reference only has to follow the true maximum from
    // afar: on most tiles nothing moves, no maximum is worked out and O^T is left alone.
    auto exceeds = [&](const float (&v)[KC]) -> bool {
      bool exceed = false;
#pragma unroll
      for (int c = 0; c < KC / 8; ++c)
        if (c < nch) {
          const float4 ta = *reinterpret_cast<const float4*>(w_thr + 8 * c), tb = *reinterpret_cast<const float4*>(w_thr + 8 * c + 4);
          exceed = exceed || v[8 * c] > ta.x || v[8 * c + 1] > ta.y || v[8 * c + 2] > ta.z || v[8 * c + 3] > ta.w ||
                   v[8 * c + 4] > tb.x || v[8 * c + 5] > tb.y || v[8 * c + 6] > tb.z || v[8 * c + 7] > tb.w;
        }
      return exceed;
    };
    // tile t's P^T buffer was last read by the P V product of tile t - pbufs
    auto pbuf_free = [&](int t) -> bool {
      return t < a.pbufs || mbar_wait(b_odone + 8 * ((t - a.pbufs) & 1), (uint32_t)((t - a.pbufs) >> 1) & 1u, s_abort, a.wait_ns);
    };
    // weights 2^(score * scale - m), this lane's share of the column sums, P^T, and the hand-over of tile t
    auto emit = [&](int t, float (&v)[KC]) {
      const int tile0 = (split + t * a.nsplit) * kTileKeys;
      uint8_t* prow = sP + (size_t)(t % a.pbufs) * pbuf + (size_t)row * 128;
#pragma unroll
      for (int c = 0; c < KC / 8; ++c)
        if (c < nch) {
          const float4 na = *reinterpret_cast<const float4*>(w_nme + 8 * c), nb = *reinterpret_cast<const float4*>(w_nme + 8 * c + 4);
          const float nm[8] = {na.x, na.y, na.z, na.w, nb.x, nb.y, nb.z, nb.w};
          uint32_t hw[4], lw[4];                            // 8 columns = one 16-byte chunk of this key's row of the P^T operand
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) {
            const int j = 8 * c + 2 * jj;
            float x0, x1;
            unpack2(fma2(pack2(v[j], v[j + 1]), sc2, pack2(nm[2 * jj], nm[2 * jj + 1])), x0, x1);
            const float w0 = ex2(x0), w1 = ex2(x1);         // masked scores are -inf: weight 0
            const f32x2 w2 = pack2(w0, w1);
            lsum[j >> 1] = add2(lsum[j >> 1], w2);
            // leading bf16 terms and the bf16 terms of what that rounding lost
            const __nv_bfloat162 h = __floats2bfloat162_rn(w0, w1);
            hw[jj] = *reinterpret_cast<const uint32_t*>(&h);
            float r0, r1;
            unpack2(sub2(w2, pack2(__uint_as_float(hw[jj] << 16), __uint_as_float(hw[jj] & 0xffff0000u))), r0, r1);
            const __nv_bfloat162 l = __floats2bfloat162_rn(r0, r1);
            lw[jj] = *reinterpret_cast<const uint32_t*>(&l);
          }
          const int ch = (q0 >> 3) + c, cl = ch + (NQ >> 3);   // chunk index over all 2 NQ columns: leading terms, trailing terms
          *reinterpret_cast<uint4*>(prow + (size_t)(ch >> 3) * kHalfBytes + ((((uint32_t)ch & 7u) ^ ((uint32_t)row & 7u)) << 4)) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
          *reinterpret_cast<uint4*>(prow + (size_t)(cl >> 3) * kHalfBytes + ((((uint32_t)cl & 7u) ^ ((uint32_t)row & 7u)) << 4)) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
        }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      // keys past the longest row of this sequence hold whatever the cache held: zero their V rows
      if (tile0 + kTileKeys > lmax) {
        const int s = t % vstages;
        if (!mbar_wait(b_vfull + 8 * s, (uint32_t)(t / vstages) & 1u, s_abort, a.wait_ns)) *s_abort = 1;
        uint8_t* vs = sV + (size_t)s * 2 * kHalfBytes;
        for (int rr = max(lmax - tile0, 0) + (warp * 32 + lane); rr < kTileKeys; rr += kSoftThreads) {
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            *reinterpret_cast<uint4*>(vs + (size_t)rr * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(vs + kHalfBytes + (size_t)rr * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(b_pready + 8 * (t & 1));
    };
    // With four S^T buffers the tiles are taken two at a time: one wait for both score products, one
    // vote, then the two sets of weights back to back - half the hand-overs per key.  When the vote
    // says that a reference point has to move, the tile is finished on its own and the next turn
    // starts with its neighbour.
    for (int i = 0; i < ntl;) {
      const int sp = i & 1;
      const bool pair = NSB == 4 && i + 1 < ntl;
      float v[KC], v_next[NSB == 4 ? KC : 1];
      bool ok = load_scores(i, v);
      bool exceed = exceeds(v);
      if constexpr (NSB == 4) {
        if (pair) {
          ok = load_scores(i + 1, v_next) && ok;
          exceed = exceed || exceeds(v_next);
        }
      }
      ok = pbuf_free(i) && ok;
      const bool bad = !ok || *s_abort != 0;
      const bool moved = group_any(1 + grp, exceed || bad);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");   // (the waits above order the reads of O^T below)
      if (moved) {
        // ---- the rare path: the true maxima of the tile, new reference points where needed
        if (!group_all(1 + grp, !bad)) { *s_abort = 1; have = false; break; }   // the same decision in every thread of the group
        float* red_w = s_red + (sp * kSoftWarps + warp) * kCols;
        {
          float x[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) x[j] = (j < KC && j < ncol) ? v[j < KC ? j : 0] : -INFINITY;
          const float r = warp_max32(x, lane);
          if (lane < ncol) red_w[lane] = r;
        }
        group_all(1 + grp, true);
        const float* red = s_red + (sp * kSoftWarps + grp * 4) * kCols;
        // lane j works column j out; the other lanes get the factors by shuffle
        float mnA = -INFINITY, crA = 1.f;
        bool mvA = false;
        if (lane < ncol && q0 + lane < nq) {
          const float t = fmaxf(fmaxf(red[lane], red[kCols + lane]), fmaxf(red[2 * kCols + lane], red[3 * kCols + lane])) * sc;
          const float mo = w_mo[lane];                   // (sc > 0: scaling commutes with the maximum)
          mvA = (mo == -INFINITY) ? (t > mo) : (t > mo + 8.f);
          mnA = mvA ? t : mo;
          crA = mvA ? ((mo == -INFINITY) ? 0.f : ex2(mo - t)) : 1.f;
        }
        const unsigned grewA = __ballot_sync(0xffffffffu, mvA);
        bool prev_done = a.pbufs == 1;                   // is the P V product of tile i - 1 known to have retired?
#pragma unroll
        for (int c = 0; c < KC / 8; ++c) {
          if (c < nch) {
            const bool grew = ((grewA >> (8 * c)) & 0xffu) != 0;   // the same in every thread of the group
            if (grew) {
              float cr[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                cr[j] = __shfl_sync(0xffffffffu, crA, 8 * c + j);
                if (j & 1) {
                  float s0, s1;
                  unpack2(lsum[(8 * c + j) >> 1], s0, s1);
                  lsum[(8 * c + j) >> 1] = pack2(s0 * cr[j - 1], s1 * cr[j]);
                }
              }
              if (i > 0) {
                if (!prev_done) {                        // O^T must hold all of tile i - 1 before it is rescaled
                  if (!mbar_wait(b_odone + 8 * ((i - 1) & 1), (uint32_t)((i - 1) >> 1) & 1u, s_abort, a.wait_ns)) *s_abort = 1;
                  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                  prev_done = true;
                }
#pragma unroll
                for (int t = 0; t < 2; ++t) {            // the shares of both weight terms
                  float o[8];
                  tmem_ld8_nowait(lane_base + ocol + (uint32_t)(t * NQ + q0 + 8 * c), o);
                  tmem_ld_wait();
                  tmem_landed8(o);
#pragma unroll
                  for (int j = 0; j < 8; ++j) o[j] *= cr[j];
                  tmem_st8(lane_base + ocol + (uint32_t)(t * NQ + q0 + 8 * c), o);
                }
              }
            }
          }
        }
        __syncwarp();
        if (lane < ncol && q0 + lane < nq) {
          w_mo[lane] = mnA;
          w_thr[lane] = (mnA + 8.f) / sc;
          w_nme[lane] = (mnA == -INFINITY) ? -INFINITY : -mnA;
        }
        __syncwarp();
              emit(i, v);
        i += 1;
        continue;
      }
      emit(i, v);
      if constexpr (NSB == 4) {
        if (pair) {
          if (!pbuf_free(i + 1)) *s_abort = 1;
          emit(i + 1, v_next);
        }
      }
      i += pair ? 2 : 1;
    }
    // ---- un-normalised result of this key slice
    if (have) {
      bool ok = mbar_wait(b_odone + 8 * ((ntl - 1) & 1), (uint32_t)((ntl - 1) >> 1) & 1u, s_abort, a.wait_ns);
      ok = group_all(1 + grp, ok && *s_abort == 0);
      if (!ok) { *s_abort = 1; have = false; }
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // O^T: this thread holds head dim `row` of its columns; one 512-byte row of the partial output per column
#pragma unroll
    for (int c = 0; c < KC / 8; ++c) {
      if (c < nch) {
        float o[8];
        if (have) {
          float w[8];
          tmem_ld8_nowait(lane_base + ocol + (uint32_t)(q0 + 8 * c), o);
          tmem_ld8_nowait(lane_base + ocol + (uint32_t)(NQ + q0 + 8 * c), w);
          tmem_ld_wait();
          tmem_landed8(o);
          tmem_landed8(w);
#pragma unroll
          for (int j = 0; j < 8; ++j) o[j] += w[j];
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) o[j] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int q = q0 + 8 * c + j;
          if (q < nq) {
            const size_t obase = ((size_t)split * a.rows + (b * R + r0 + q / G)) * a.H + (kvh * G + q % G);
            a.out_o[obase * kDh + row] = o[j];
          }
        }
      }
    }
    // the column sums: add the 128 key lanes' shares up (warp shuffle, then the four warps of the group)
    float* sum_w = s_red + warp * kCols;
#pragma unroll
    for (int c = 0; c < KC / 8; ++c) {
      if (c < nch) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          float t, t_other;
          if (j & 1) unpack2(lsum[(8 * c + j) >> 1], t_other, t); else unpack2(lsum[(8 * c + j) >> 1], t, t_other);
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
          if (lane == 0) sum_w[8 * c + j] = t;
        }
      }
    }
    group_all(1 + grp, true);
    if (wq == 0) {
      const float* red = s_red + (grp * 4) * kCols;
      const float* m_fin = w_mo;                       // (warp 4 * grp: its own copy)
      constexpr float kLn2 = 0.6931471805599453f;
      for (int col = lane; col < ncol; col += 32) {
        const int q = q0 + col;
        if (q < nq) {
          const float l = (red[col] + red[kCols + col]) + (red[2 * kCols + col] + red[3 * kCols + col]);
          const size_t obase = ((size_t)split * a.rows + (b * R + r0 + q / G)) * a.H + (kvh * G + q % G);
          a.out_ml[obase * 2] = have ? m_fin[col] * kLn2 : -INFINITY;
          a.out_ml[obase * 2 + 1] = have ? l : 0.f;
        }
      }
    }
    if (*s_abort && lane == 0) atomicOr(a.status, CS_DEV_TIMEOUT);
  }
  // ---------------------------------------------------------------------- teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (tid == 0) cs_stamp_end(a.stamp);
  if (warp == kMmaWarp) {
    if (*s_abort && lane == 0 && ntl > 0) mbar_wait(b_odone + 8 * ((ntl - 1) & 1), (uint32_t)((ntl - 1) >> 1) & 1u, s_never, a.wait_ns);   // MMAs retired (bounded)
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

}  // namespace

int cs_launch_attention_tcw(cs_ctx* ctx, const void* kv_cache, int layer, int B, int R, cudaStream_t st) {
  const cs_model_config& c = ctx->cfg;
  const int G = c.n_heads / c.n_kv_heads;
  if (c.head_dim != kDh || G > kNQMax || R < 1 || R > 256) return 0;
  // blocks with more than 96 query rows per KV head are cut into groups of block rows
  const int ngroups = cs_ceil_div(G * R, kNQMax), Rg = cs_ceil_div(R, ngroups);
  if (G * Rg > kNQMax) return 0;
  const int nq = G * Rg;
  const int NQ = (nq + 23) / 24 * 24;                  // three column groups of whole 8-column chunks
  if (ctx->tmKV_base != kv_cache) {
    const unsigned long long rows = (unsigned long long)c.n_layers * 2 * c.max_batch * c.n_kv_heads * c.max_seq;
    if (rows > 0x7fffffffull) return 0;
    const unsigned long long dims[2] = {(unsigned long long)kDh, rows}, strides[1] = {kDh * 2};
    const unsigned box[2] = {64, (unsigned)kTileKeys};
    if (cs_encode_tiled(ctx, &ctx->tmKV, kv_cache, 2, dims, strides, box) != CS_OK) return -1;
    ctx->tmKV_base = kv_cache;
  }
  if (ctx->tmQ_R != Rg) {
    const unsigned long long dims[3] = {(unsigned long long)kDh, (unsigned long long)c.n_heads, 2ull * CS_MAX_ROWS};
    const unsigned long long strides[2] = {kDh * 2, (unsigned long long)c.n_heads * kDh * 2};
    const unsigned box[3] = {64, (unsigned)G, (unsigned)Rg};
    if (cs_encode_tiled(ctx, &ctx->tmQ, ctx->qbuf, 3, dims, strides, box) != CS_OK) return -1;
    ctx->tmQ_R = Rg;
  }
  // one CTA per SM: Q (two terms), P^T (two terms, 64-column atoms), two K stages, one or two V stages,
  // then barriers, flags and the softmax scratch; 1 KB of slack for the 1024-byte alignment
  const size_t natoms = (size_t)(2 * NQ + 63) / 64;
  const size_t base = 1024 + (size_t)4 * NQ * 128 + (size_t)2 * 2 * kHalfBytes;
  const size_t pbuf = natoms * kHalfBytes, vstage = (size_t)2 * kHalfBytes;
  const size_t ctl = (size_t)kCtlBytes + kNQMax * 4 + kSoftWarps * 3 * kCols * 4 + 2 * kSoftWarps * kCols * 4;
  const size_t limit = 227 * 1024;
  // in order of what it buys: a second P^T buffer (the softmax no longer waits for the previous
  // tile's P V product), then a second V stage
  const int pbufs = (base + 2 * pbuf + vstage + ctl <= limit) ? 2 : 1;
  const int vstages = (base + pbufs * pbuf + 2 * vstage + ctl <= limit) ? 2 : 1;
  const size_t smem = base + pbufs * pbuf + vstages * vstage + ctl;
  if (smem > limit) return 0;
  int nsplit = ctx->num_sms / (B * c.n_kv_heads * ngroups);
  if (nsplit > ctx->attn_splits) nsplit = ctx->attn_splits;
  if (nsplit < 1) nsplit = 1;
  // up to 48 query rows (16 columns per softmax thread) with two P^T buffers: four S^T buffers, tiles in pairs
  const bool dual = NQ <= 48 && pbufs == 2;
  auto kernel = dual ? k_attn_tcw<16, 4> : k_attn_tcw<kCols, 2>;
  if (smem > ctx->attn_tcw_smem_set) {                 // (both instantiations are raised together: one high-water mark)
    if (cudaFuncSetAttribute(k_attn_tcw<16, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(k_attn_tcw<kCols, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
      snprintf(ctx->err, sizeof(ctx->err), "attention needs %zu bytes of shared memory", smem);
      return -1;
    }
    ctx->attn_tcw_smem_set = smem;
  }
  AttnArgs a;
  a.row_lim = ctx->row_lim;
  a.kv_len_early = ctx->kv_len_early;
  a.layer = layer; a.R = R; a.Rg = Rg; a.G = G; a.H = c.n_heads; a.Hkv = c.n_kv_heads;
  a.max_batch = c.max_batch; a.max_seq = c.max_seq; a.nsplit = nsplit; a.NQ = NQ; a.rows = B * R; a.vstages = vstages; a.pbufs = pbufs;
  a.qstack = (3 * ((2 * NQ + 31) / 32 * 32) <= 512) ? 1 : 0;   // TMEM columns: two score buffers and the output, 2 NQ wide each
  if (dual && 5 * ((2 * NQ + 31) / 32 * 32) > 512) return 0;   // (four score buffers and the output: 480 columns at 48 query rows)
  a.smem_bytes = (int)smem;
  a.scale_log2e = 1.4426950408889634f / sqrtf((float)kDh);
  a.out_o = ctx->attn_o; a.out_ml = ctx->attn_ml; a.status = ctx->d_status;
  a.wait_ns = ctx->wait_limit_ns;
  a.stamp = cs_next_stamp(ctx, CS_FAM_ATTENTION);
  if (cs_launch_pdl(kernel, dim3(B * c.n_kv_heads, nsplit, ngroups), dim3(kThreads), smem, st, ctx->tmKV, ctx->tmQ, a) != cudaSuccess) {
    snprintf(ctx->err, sizeof(ctx->err), "attention launch failed");
    return -1;
  }
  return nsplit;
}
