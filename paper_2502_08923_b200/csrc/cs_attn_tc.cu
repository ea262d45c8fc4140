// Causal block attention over the bf16 KV cache on the 5th-generation tensor cores
// (Sec. 3.2; App. B.2), for head_dim 128.  Up to 128 query rows per KV head form one query
// tile; taller blocks are cut into groups of block rows, one group per CTA.
//
// One CTA = one (sequence, KV head) and one slice of the key range.  The query rows (the
// (k+1) block rows of the G query heads sharing the KV head) are the M dimension of both
// products, so that TMEM lane i belongs to query row i and the online softmax of a row is
// shared by just two threads (warps w and w + 4 both reach TMEM lanes 32 w .. 32 w + 31; one
// takes keys 0-63 of a tile and output dims 0-63, the other the upper halves; they exchange
// their row maxima and sums through shared memory and a bounded mbarrier wait):
//     S [128 x 128 keys]  = Q_hi K_tile^T + Q_lo K_tile^T     (tcgen05.mma, A and B K-major)
//     O [128 x 128 dims] += P_hi V_tile  + P_lo V_tile        (tcgen05.mma, B MN-major)
// Queries and softmax weights enter as two bf16 terms each, so they are fp32-equivalent and
// only K and V - which the cache stores in bf16 - are rounded.  Only the first nq of the 128
// rows are real: the A-operand buffers hold just those rows and the MMAs read on into the
// shared memory behind them; whatever they find there only reaches accumulator rows that
// nobody reads.  K and V tiles arrive by TMA (128-byte swizzle, two 64-wide halves) through
// an mbarrier ring.  Each CTA writes its un-normalised (O, max, sum); k_attn_merge combines
// the slices.  A K buffer is handed back to the producer as soon as the score product that
// read it has retired and a V buffer after the P V product, so with a single stage the next
// tile's K lands during the softmax and its V during the next score product.  When the caller
// vouches for the cached lengths (kv_len_early), a slice whose first tile lies wholly below
// the cached length requests that tile before it waits for the preceding kernel: those rows
// were written by earlier steps.  Every wait is bounded (2 s by default): on expiry the CTA flags
// CS_DEV_TIMEOUT, drains its copies, frees its TMEM and returns.
#include <stdlib.h>

#include "cs_common.cuh"

namespace {

constexpr int kThreads = 320;   // warps 0-7 softmax/epilogue, warp 8 TMA producer, warp 9 MMA
constexpr int kProdWarp = 8, kMmaWarp = 9;
constexpr int kCtlBytes = 160;  // 16 mbarriers + TMEM slot + flags
constexpr int kTileKeys = 128;
constexpr int kDh = 128;
constexpr int kHalfBytes = kTileKeys * 128;          // one [128 keys x 64 dims] half tile
constexpr int kNQMax = 128;

struct AttnArgs {
  const int* row_lim;
  const int* kv_len_early;   // cached lengths that no kernel in flight changes, or NULL
  int layer, R, Rg, G, H, Hkv, max_batch, max_seq, nsplit, NQ, rows, stages;   // Rg = block rows per row group
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]) :: "memory");   // the registers are valid only from here on
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// 32 accumulator columns with one wait (two loads in flight)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr + 16u));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
  asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]) :: "memory");   // the registers are valid only from here on
  asm volatile("" : "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31]) :: "memory");   // the registers are valid only from here on
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// 2^x, hardware approximation (relative error about 2^-22; -inf gives 0)
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
        "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
        "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15]))
      : "memory");
}
// eight values as eight leading bf16 terms and the eight bf16 terms of what that rounding lost
__device__ __forceinline__ void split8(const float* p, uint4& hi, uint4& lo) {
  uint32_t h[4], l[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(p[2 * i], p[2 * i + 1]);
    const float2 af = __bfloat1622float2(a);
    const __nv_bfloat162 b = __floats2bfloat162_rn(p[2 * i] - af.x, p[2 * i + 1] - af.y);
    h[i] = *reinterpret_cast<const uint32_t*>(&a);
    l[i] = *reinterpret_cast<const uint32_t*>(&b);
  }
  hi = make_uint4(h[0], h[1], h[2], h[3]);
  lo = make_uint4(l[0], l[1], l[2], l[3]);
}

__global__ void __launch_bounds__(kThreads, 2)
k_attn_tc(const __grid_constant__ CUtensorMap tmKV, const __grid_constant__ CUtensorMap tmQ, AttnArgs a) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  // blockIdx.z picks a group of Rg consecutive block rows (blocks taller than 128 / G rows)
  const int NQ = a.NQ, G = a.G, R = a.R, r0 = blockIdx.z * a.Rg, Rcur = min(a.Rg, R - r0);
  const int nq = G * Rcur, nq_box = G * a.Rg, stages = a.stages;
  const uint32_t qhalf = (uint32_t)NQ * 128u;          // [NQ rows x 64 elements] of one term
  const uint32_t qterm = 2u * qhalf;
  // A operands first, K/V behind them: the MMAs' reads past row NQ stay inside the allocation
  uint8_t* sQ = smem;                                  // [term][half][NQ][128 B]
  uint8_t* sP = sQ + 2 * qterm;                        // same shape, 64 keys per half
  uint8_t* sK = sP + 2 * qterm;                        // [stage][half][128 keys][128 B]
  uint8_t* sV = sK + (size_t)stages * 2 * kHalfBytes;
  // Barriers, flags and the exchange rows of the softmax pairs (two parities x two halves x NQ
  // floats) live in what the 1024-byte alignment leaves over: in front of the aligned area when
  // that holds them, else behind it.  (The window normally starts aligned, so they sit behind.)
  uint8_t* tail = sV + (size_t)stages * 2 * kHalfBytes;
  const uint32_t pad = (uint32_t)(smem - smem_raw), need = (uint32_t)kCtlBytes + 16u * (uint32_t)NQ;
  const uint32_t back = (uint32_t)a.smem_bytes - pad - (uint32_t)(tail - smem);
  if (pad < need && back < need) {   // cannot happen with the sizes the launcher asks for unless the window starts oddly
    if (threadIdx.x == 0) atomicOr(a.status, CS_DEV_SMEM);
    return;
  }
  uint64_t* bars = reinterpret_cast<uint64_t*>(pad >= need ? smem_raw : tail);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* s_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_never = reinterpret_cast<volatile int*>(tmem_slot + 2);
  int* s_lmax = reinterpret_cast<int*>(tmem_slot + 3);
  float* s_xch = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + kCtlBytes);   // [parity][half][NQ]
  const uint32_t b_kfull = smem_u32(bars), b_vfull = smem_u32(bars + 2), b_kfree = smem_u32(bars + 4),
                 b_vfree = smem_u32(bars + 6), b_qfull = smem_u32(bars + 8), b_sready = smem_u32(bars + 9),
                 b_pready = smem_u32(bars + 10), b_odone = smem_u32(bars + 11), b_pair = smem_u32(bars + 12);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.x / a.Hkv, kvh = blockIdx.x % a.Hkv, split = blockIdx.y;
  const int nact = (nq + 31) >> 5;                     // softmax warps that own real rows
  constexpr uint32_t kTmemCols = 256, kOCol = 128;     // S in columns 0..127, O in 128..255

  if (tid == kProdWarp * 32) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(b_kfull + 8 * s, 1); mbar_init(b_vfull + 8 * s, 1);
      mbar_init(b_kfree + 8 * s, 1); mbar_init(b_vfree + 8 * s, 1);
    }
    mbar_init(b_qfull, 1);
    mbar_init(b_sready, 1);
    mbar_init(b_pready, (uint32_t)nact * 64u);
    mbar_init(b_odone, 1);
    for (int w = 0; w < 4; ++w) mbar_init(b_pair + 8 * w, 64);
    *s_abort = 0; *s_never = 0; *s_lmax = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmKV) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmQ) : "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  // Slice `split` works on key tiles split, split + nsplit, ...: its first tile is known before
  // the key range is, so the queries and that tile are requested while the range is worked out
  // (a slice beyond the range only has to let them land).
  const long long krow = ((((long long)a.layer * 2 + 0) * a.max_batch + b) * a.Hkv + kvh) * (long long)a.max_seq;
  const long long vrow = ((((long long)a.layer * 2 + 1) * a.max_batch + b) * a.Hkv + kvh) * (long long)a.max_seq;
  const int key_first = split * kTileKeys;
  bool early = false;
  if (warp == kProdWarp && lane == 0 && a.kv_len_early != nullptr) {
    // a tile of cached keys only: nothing in flight writes it, so it need not wait
    if (key_first + kTileKeys <= min(a.kv_len_early[b], a.max_seq)) {
      early = true;
      const uint32_t dk = smem_u32(sK), dv = smem_u32(sV);
      mbar_expect_tx(b_kfull, 2u * kHalfBytes);
      tma_load_2d(dk, &tmKV, b_kfull, 0, (int)(krow + key_first));
      tma_load_2d(dk + kHalfBytes, &tmKV, b_kfull, 64, (int)(krow + key_first));
      mbar_expect_tx(b_vfull, 2u * kHalfBytes);
      tma_load_2d(dv, &tmKV, b_vfull, 0, (int)(vrow + key_first));
      tma_load_2d(dv + kHalfBytes, &tmKV, b_vfull, 64, (int)(vrow + key_first));
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp < 8) {
    int lm = 0;
    for (int r = tid; r < Rcur; r += 256) lm = max(lm, a.row_lim[b * R + r0 + r]);
    lm = __reduce_max_sync(0xffffffffu, lm);
    if (lane == 0 && lm > 0) atomicMax(s_lmax, lm);
  }
  if (warp == kProdWarp && lane == 0) {
    // K first (it comes from HBM and the first product waits for it), then the queries (fresh in
    // L2), V last: it is not needed before the softmax of the tile is done
    const uint32_t dk = smem_u32(sK), dv = smem_u32(sV);
    if (!early) {
      mbar_expect_tx(b_kfull, 2u * kHalfBytes);
      tma_load_2d(dk, &tmKV, b_kfull, 0, (int)(krow + key_first));
      tma_load_2d(dk + kHalfBytes, &tmKV, b_kfull, 64, (int)(krow + key_first));
    }
    mbar_expect_tx(b_qfull, (uint32_t)(4 * nq_box * 128));
    for (int term = 0; term < 2; ++term)
      for (int dh = 0; dh < 2; ++dh)
        tma_load_3d(smem_u32(sQ + term * qterm + dh * qhalf), &tmQ, b_qfull, dh * 64, kvh * G,
                    term * CS_MAX_ROWS + b * R + r0);   // the box is always Rg rows tall; rows past the group are never used
    if (!early) {
      mbar_expect_tx(b_vfull, 2u * kHalfBytes);
      tma_load_2d(dv, &tmKV, b_vfull, 0, (int)(vrow + key_first));
      tma_load_2d(dv + kHalfBytes, &tmKV, b_vfull, 64, (int)(vrow + key_first));
    }
  }
  __syncthreads();
  const int lmax = *s_lmax;
  const int ntiles = (lmax + kTileKeys - 1) / kTileKeys;
  const int ntl = (ntiles > split) ? (ntiles - split + a.nsplit - 1) / a.nsplit : 0;

  if (warp == kProdWarp) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int ik = 1, iv = 1;   // K and V tiles requested so far (tile 0 of this slice is already on its way)
      bool ok = true;
      for (int i = 1; i < ntl; ++i) {
        const int s = i % stages;
        const uint32_t ph = (uint32_t)(i / stages) & 1u;
        const int key0 = (split + i * a.nsplit) * kTileKeys;
        const uint32_t dk = smem_u32(sK + (size_t)s * 2 * kHalfBytes), dv = smem_u32(sV + (size_t)s * 2 * kHalfBytes);
        if (!mbar_wait(b_kfree + 8 * s, ph ^ 1u, s_abort, a.wait_ns)) { ok = false; break; }
        mbar_expect_tx(b_kfull + 8 * s, 2u * kHalfBytes);
        tma_load_2d(dk, &tmKV, b_kfull + 8 * s, 0, (int)(krow + key0));
        tma_load_2d(dk + kHalfBytes, &tmKV, b_kfull + 8 * s, 64, (int)(krow + key0));
        ik = i + 1;
        if (!mbar_wait(b_vfree + 8 * s, ph ^ 1u, s_abort, a.wait_ns)) { ok = false; break; }
        mbar_expect_tx(b_vfull + 8 * s, 2u * kHalfBytes);
        tma_load_2d(dv, &tmKV, b_vfull + 8 * s, 0, (int)(vrow + key0));
        tma_load_2d(dv + kHalfBytes, &tmKV, b_vfull + 8 * s, 64, (int)(vrow + key0));
        iv = i + 1;
      }
      if (!ok) { *s_abort = 1; atomicOr(a.status, CS_DEV_TIMEOUT); }
      if (*s_abort || ntl == 0) {   // let the copies land before the shared memory goes away
        mbar_wait(b_qfull, 0, s_never, a.wait_ns);
        for (int j = max(0, ik - stages); j < ik; ++j) mbar_wait(b_kfull + 8 * (j % stages), (uint32_t)(j / stages) & 1u, s_never, a.wait_ns);
        for (int j = max(0, iv - stages); j < iv; ++j) mbar_wait(b_vfull + 8 * (j % stages), (uint32_t)(j / stages) & 1u, s_never, a.wait_ns);
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && ntl > 0) {
      const uint32_t idesc1 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
      const uint32_t idesc2 = idesc1 | (1u << 16);      // B (= V) is MN-major
      const uint32_t aq = smem_u32(sQ), ap = smem_u32(sP);
      // S of tile i: issued behind the P V product of tile i - 1, so one commit covers both
      auto issue_scores = [&](int i) -> bool {
        const int s = i % stages;
        if (!mbar_wait(b_kfull + 8 * s, (uint32_t)(i / stages) & 1u, s_abort, a.wait_ns)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t ak = smem_u32(sK + (size_t)s * 2 * kHalfBytes);
#pragma unroll
        for (int term = 0; term < 2; ++term)
#pragma unroll
          for (int dh = 0; dh < 2; ++dh)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              umma_bf16(tmem_base, desc_kmajor(aq + term * qterm + dh * qhalf) + 2 * kk, desc_kmajor(ak + dh * kHalfBytes) + 2 * kk,
                        idesc1, (term | dh | kk) ? 1u : 0u);
        umma_commit(b_kfree + 8 * s);
        umma_commit(b_sready);
        return true;
      };
      bool ok = mbar_wait(b_qfull, 0, s_abort, a.wait_ns) && issue_scores(0);
      for (int i = 0; i < ntl && ok; ++i) {
        const int s = i % stages;
        const uint32_t ph = (uint32_t)(i / stages) & 1u;
        if (!mbar_wait(b_pready, (uint32_t)i & 1u, s_abort, a.wait_ns) || !mbar_wait(b_vfull + 8 * s, ph, s_abort, a.wait_ns)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t av = smem_u32(sV + (size_t)s * 2 * kHalfBytes);
#pragma unroll
        for (int term = 0; term < 2; ++term)
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)   // 16 keys per instruction
            umma_bf16(tmem_base + kOCol, desc_kmajor(ap + term * qterm + (kk >> 2) * qhalf) + 2 * (kk & 3),
                      desc_mnmajor(av + kk * 2048, kHalfBytes), idesc2, (i > 0 || term > 0 || kk > 0) ? 1u : 0u);
        umma_commit(b_vfree + 8 * s);
        umma_commit(b_odone);
        if (i + 1 < ntl && !issue_scores(i + 1)) { ok = false; break; }
      }
      if (!ok) { *s_abort = 1; atomicOr(a.status, CS_DEV_TIMEOUT); }
    }
  } else if ((warp & 3) < nact) {
    // ------------------------------------------------------------------ softmax + epilogue (two threads per query row)
    const int wq = warp & 3, half = warp >> 2;
    const int q = wq * 32 + lane;
    const bool valid = q < nq;
    const int lim = valid ? a.row_lim[b * R + r0 + q / G] : 0;
    const uint32_t lane_base = tmem_base + ((uint32_t)(wq * 32) << 16);
    const uint32_t col0 = (uint32_t)half * 64u;        // this thread's keys of a tile and its output dims
    const uint32_t pairbar = b_pair + 8u * (uint32_t)wq;
    const float sc = a.scale_log2e;
    float m = -INFINITY, l = 0.f;                      // running max (log2 domain, whole row) and sum of this half
    bool have = ntl > 0;
    uint32_t xuse = 0;                                 // exchanges done so far
    // hand `mine` to the other thread of the row and return what it handed over
    auto exchange = [&](float mine, float& theirs) -> bool {
      float* slot = s_xch + (size_t)(xuse & 1u) * 2 * NQ;
      if (valid) slot[half * NQ + q] = mine;
      mbar_arrive(pairbar);
      const bool ok = mbar_wait(pairbar, xuse & 1u, s_abort, a.wait_ns);
      theirs = (ok && valid) ? slot[(half ^ 1) * NQ + q] : mine;
      ++xuse;
      return ok;
    };
    for (int i = 0; i < ntl; ++i) {
      const int s = i % stages;
      const uint32_t ph = (uint32_t)(i / stages) & 1u;
      const int key0 = (split + i * a.nsplit) * kTileKeys + (int)col0;   // first key of this thread's half tile
      // (S of this tile complete also means the previous tile's P V product has retired:
      //  P may be overwritten and O is up to date)
      bool ok = mbar_wait(b_sready, (uint32_t)i & 1u, s_abort, a.wait_ns);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { *s_abort = 1; have = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float mx = -INFINITY;
      const bool whole = key0 + 64 <= lim;             // no key of this half tile is masked for this row
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        float v[32];
        tmem_ld32(lane_base + col0 + (uint32_t)(c * 32), v);
        if (whole) {
#pragma unroll
          for (int j = 0; j < 32; ++j) mx = fmaxf(mx, v[j]);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (key0 + c * 32 + j < lim) mx = fmaxf(mx, v[j]);
        }
      }
      float mx_other;
      ok = exchange(mx, mx_other);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { *s_abort = 1; have = false; break; }
      mx = fmaxf(mx, mx_other) * sc;                   // sc > 0: scaling commutes with the maximum
      const float m_new = fmaxf(m, mx);
      const float corr = (m == -INFINITY) ? 0.f : ex2(m - m_new);
      if (i > 0 && __any_sync(0xffffffffu, m_new > m)) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float o[16];
          tmem_ld16(lane_base + kOCol + col0 + (uint32_t)(c * 16), o);
#pragma unroll
          for (int j = 0; j < 16; ++j) o[j] *= corr;
          tmem_st16(lane_base + kOCol + col0 + (uint32_t)(c * 16), o);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      }
      l *= corr;
      m = m_new;
      uint8_t* prow = sP + (size_t)half * qhalf + (size_t)q * 128;
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        float v[32];
        tmem_ld32(lane_base + col0 + (uint32_t)(c * 32), v);
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          v[j] = (whole || key0 + c * 32 + j < lim) ? ex2(fmaf(v[j], sc, -m_new)) : 0.f;
          l += v[j];
        }
        if (valid) {
#pragma unroll
          for (int h = 0; h < 4; ++h) {      // 8 keys = one 16-byte chunk of the operand row
            uint4 hi, lo;
            split8(v + 8 * h, hi, lo);
            const uint32_t off = (((uint32_t)(4 * c + h)) ^ ((uint32_t)q & 7u)) << 4;
            *reinterpret_cast<uint4*>(prow + off) = hi;
            *reinterpret_cast<uint4*>(prow + qterm + off) = lo;
          }
        }
      }
      // keys past the longest row of this sequence hold whatever the cache held: zero their V rows
      const int tile0 = key0 - (int)col0;
      if (tile0 + kTileKeys > lmax) {
        if (!mbar_wait(b_vfull + 8 * s, ph, s_abort, a.wait_ns)) *s_abort = 1;
        uint8_t* vs = sV + (size_t)s * 2 * kHalfBytes;
        for (int rr = max(lmax - tile0, 0) + half * nact * 32 + q; rr < kTileKeys; rr += nact * 64) {
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            *reinterpret_cast<uint4*>(vs + (size_t)rr * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(vs + kHalfBytes + (size_t)rr * 128 + c * 16) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(b_pready);
    }
    // ---- un-normalised result of this key slice
    if (have) {
      bool ok = mbar_wait(b_odone, (uint32_t)(ntl - 1) & 1u, s_abort, a.wait_ns);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { *s_abort = 1; have = false; }
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const size_t obase = valid ? ((size_t)split * a.rows + (b * R + r0 + q / G)) * a.H + (kvh * G + q % G) : 0;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      float o[16];
      if (have) {
        tmem_ld16(lane_base + kOCol + col0 + (uint32_t)(c * 16), o);
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) o[j] = 0.f;
      }
      if (valid) {
        float4* dst = reinterpret_cast<float4*>(a.out_o + obase * kDh + col0 + c * 16);
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[j] = make_float4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
      }
    }
    // the row's sum is the sum of its two halves (both are relative to the same maximum)
    float l_other = 0.f;
    if (have) {
      bool ok = exchange(l, l_other);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) { *s_abort = 1; have = false; }
    }
    if (valid && half == 0) {
      constexpr float kLn2 = 0.6931471805599453f;
      a.out_ml[obase * 2] = have ? m * kLn2 : -INFINITY;
      a.out_ml[obase * 2 + 1] = have ? l + l_other : 0.f;
    }
    if (*s_abort && lane == 0) atomicOr(a.status, CS_DEV_TIMEOUT);
  }
  // ---------------------------------------------------------------------- teardown
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (tid == 0) cs_stamp_end(a.stamp);
  if (warp == kMmaWarp) {
    if (*s_abort && lane == 0 && ntl > 0) mbar_wait(b_odone, (uint32_t)(ntl - 1) & 1u, s_never, a.wait_ns);   // MMAs retired (bounded)
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

}  // namespace

// Key tiles a CTA of this kernel walks at most for a block of B x R rows (same launch arithmetic as
// below): the dispatcher hands longer walks to the kernel with keys and head dims as M.
int cs_attention_tc_tiles_per_cta(const cs_ctx* ctx, int B, int R) {
  const cs_model_config& c = ctx->cfg;
  const int G = c.n_heads / c.n_kv_heads;
  if (c.head_dim != kDh || G > kNQMax || R < 1) return 0;
  const int ngroups = cs_ceil_div(G * R, kNQMax), Rg = cs_ceil_div(R, ngroups);
  const int NQ = (G * Rg + 15) / 16 * 16;
  const bool small = 1024 + (size_t)8 * NQ * 128 + (size_t)4 * kHalfBytes <= (size_t)113 * 1024 && (size_t)kCtlBytes + 16 * (size_t)NQ <= 1024;
  int nsplit = (small ? 2 : 1) * ctx->num_sms / (B * c.n_kv_heads * ngroups);
  if (nsplit > ctx->attn_splits) nsplit = ctx->attn_splits;
  if (nsplit < 1) nsplit = 1;
  return cs_ceil_div(cs_ceil_div(c.max_seq, kTileKeys), nsplit);
}

// Query rows per KV head that one CTA of this kernel holds for a block of R rows (of its 128 M rows).
int cs_attention_tc_group_rows(const cs_ctx* ctx, int R) {
  const cs_model_config& c = ctx->cfg;
  const int G = c.n_heads / c.n_kv_heads;
  if (c.head_dim != kDh || G > kNQMax || R < 1) return 0;
  const int ngroups = cs_ceil_div(G * R, kNQMax);
  return G * cs_ceil_div(R, ngroups);
}

int cs_launch_attention_tc(cs_ctx* ctx, const void* kv_cache, int layer, int B, int R, cudaStream_t st) {
  const cs_model_config& c = ctx->cfg;
  const int G = c.n_heads / c.n_kv_heads;
  if (c.head_dim != kDh || G > kNQMax || R < 1 || R > 256) return 0;
  // blocks with more than 128 query rows per KV head are cut into groups of block rows
  const int ngroups = cs_ceil_div(G * R, kNQMax), Rg = cs_ceil_div(R, ngroups);
  if (G * Rg > kNQMax) return 0;
  const int nq = G * Rg;
  const int NQ = (nq + 15) / 16 * 16;
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
  // 1 KB of slack for the 1024-byte alignment; barriers, flags and the softmax exchange rows
  // (kCtlBytes + 16 NQ bytes) fit inside it for the small tiles, larger ones get that much more.
  // Small query tiles take one K/V stage and two CTAs per SM - short key slices, twice the
  // CTAs - larger ones two stages and the whole SM.
  const size_t ab = (size_t)8 * NQ * 128;                       // Q and P, two terms of two halves each
  const size_t two_per_sm = 113 * 1024, limit = 227 * 1024;
  const size_t ctl = (size_t)kCtlBytes + 16 * (size_t)NQ;
  const bool small = 1024 + ab + (size_t)4 * kHalfBytes <= two_per_sm && ctl <= 1024;
  const size_t extra = small ? 0 : (ctl + 127) / 128 * 128;
  const int stages = small ? 1 : ((1024 + extra + ab + (size_t)2 * 4 * kHalfBytes <= limit) ? 2 : 1);
  const size_t smem = 1024 + extra + ab + (size_t)stages * 4 * kHalfBytes;
  int nsplit = (small ? 2 : 1) * ctx->num_sms / (B * c.n_kv_heads * ngroups);
  if (nsplit > ctx->attn_splits) nsplit = ctx->attn_splits;
  if (nsplit < 1) nsplit = 1;
  if (smem > ctx->attn_tc_smem_set) {
    if (cudaFuncSetAttribute(k_attn_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
      snprintf(ctx->err, sizeof(ctx->err), "attention needs %zu bytes of shared memory", smem);
      return -1;
    }
    ctx->attn_tc_smem_set = smem;
  }
  AttnArgs a;
  a.row_lim = ctx->row_lim;
  a.kv_len_early = ctx->kv_len_early;
  a.layer = layer; a.R = R; a.Rg = Rg; a.G = G; a.H = c.n_heads; a.Hkv = c.n_kv_heads;
  a.max_batch = c.max_batch; a.max_seq = c.max_seq; a.nsplit = nsplit; a.NQ = NQ; a.rows = B * R; a.stages = stages;
  a.smem_bytes = (int)smem;
  a.scale_log2e = 1.4426950408889634f / sqrtf((float)kDh);
  a.out_o = ctx->attn_o; a.out_ml = ctx->attn_ml; a.status = ctx->d_status;
  a.wait_ns = ctx->wait_limit_ns;
  a.stamp = cs_next_stamp(ctx, CS_FAM_ATTENTION);
  if (cs_launch_pdl(k_attn_tc, dim3(B * c.n_kv_heads, nsplit, ngroups), dim3(kThreads), smem, st, ctx->tmKV, ctx->tmQ, a) != cudaSuccess) {
    snprintf(ctx->err, sizeof(ctx->err), "attention launch failed");
    return -1;
  }
  return nsplit;
}
