// Suffix-match search and draft gather (Sec. 3.1, 3.2; App. B.3 step 1).
//
// One thread-block cluster per sequence.  The CTAs of a cluster split the candidate
// start positions [0, n - 2*gamma] between them; each thread tests four consecutive
// candidates from two 128-bit loads of the history, the best position is reduced by
// warp vote / shared-memory atomics inside the CTA and through distributed shared
// memory across the cluster, and the first CTA of the cluster then copies the draft.
// No global scratch memory, no global atomics, one launch, deterministic.
#include <cooperative_groups.h>
#include <limits.h>

#include "cs_common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ int4 ld_nc_int4(const int* p) {
  return __ldg(reinterpret_cast<const int4*>(p));
}

__global__ void __launch_bounds__(kThreads)
k_find_match(const int* __restrict__ hist, const int* __restrict__ hist_len, int stride, int gamma,
             int k, int policy, int* __restrict__ match_pos, int* __restrict__ draft,
             int* __restrict__ draft_len, int* __restrict__ last_tok,
             const int* __restrict__ skip, unsigned long long* stamp) {
  CS_PDL_PROLOGUE();
  cg::cluster_group cluster = cg::this_cluster();
  const int b = blockIdx.y;
  const int rank = (int)cluster.block_rank();
  const int nblk = (int)cluster.num_blocks();
  const int tid = threadIdx.x;
  __shared__ int s_best;
  __shared__ int s_final;

  const int* h = hist + (size_t)b * stride;
  int n = hist_len[b];
  if (n > stride) n = stride;
  if (n < 0) n = 0;
  const bool dead = (skip != nullptr && skip[b] != 0);
  const int n_cand = dead ? 0 : n - 2 * gamma + 1;   // candidates p0 = 0 .. n - 2*gamma
  const bool latest = (policy == CS_MATCH_LATEST);
  const int none = latest ? -1 : INT_MAX;

  int key[CS_MAX_GAMMA];
#pragma unroll
  for (int j = 0; j < CS_MAX_GAMMA; ++j)
    key[j] = (j < gamma && n >= gamma) ? h[n - gamma + j] : -1;

  if (tid == 0) s_best = none;
  __syncthreads();

  int best = none;
  if (n_cand > 0) {
    const int per = (((n_cand + nblk - 1) / nblk) + 3) & ~3;
    const int lo = rank * per;
    const int hi = min(n_cand, lo + per);
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(h) & 15) == 0) && gamma <= 5;
    for (int p = lo + tid * 4; p < hi; p += kThreads * 4) {
      if (vec_ok && p + 8 <= stride) {
        // tokens p .. p+7 cover candidates p .. p+3 for gamma <= 5; what lies past the
        // accepted length only feeds candidates that `hi` masks off
        const int4 a = ld_nc_int4(h + p);
        const int4 c = ld_nc_int4(h + p + 4);
        const int t[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          bool eq = (p + i < hi);
#pragma unroll
          for (int j = 0; j < 5; ++j)
            if (j < gamma) eq = eq && (t[i + j] == key[j]);
          if (eq) best = latest ? max(best, p + i) : min(best, p + i);
        }
      } else {
        for (int i = 0; i < 4 && p + i < hi; ++i) {
          bool eq = true;
          for (int j = 0; j < gamma; ++j) eq = eq && (__ldg(h + p + i + j) == key[j]);
          if (eq) best = latest ? max(best, p + i) : min(best, p + i);
        }
      }
    }
  }
  // warp vote, then one shared-memory atomic per warp
  best = latest ? __reduce_max_sync(0xffffffffu, best) : __reduce_min_sync(0xffffffffu, best);
  if ((tid & 31) == 0 && best != none) {
    if (latest) atomicMax(&s_best, best); else atomicMin(&s_best, best);
  }
  __syncthreads();
  cluster.sync();
  if (rank == 0 && tid == 0) {
    int v = none;
    for (int r = 0; r < nblk; ++r) {
      const int o = *cluster.map_shared_rank(&s_best, r);
      v = latest ? max(v, o) : min(v, o);
    }
    s_final = (v == INT_MAX) ? -1 : v;
  }
  cluster.sync();   // remote shared memory stays alive until the first CTA has read it
  if (rank != 0) return;

  const int p0 = s_final;
  const int start = p0 + gamma;
  const int len = (p0 < 0) ? 0 : min(k, n - start);
  if (tid == 0) {
    match_pos[b] = p0;
    draft_len[b] = len;
    if (last_tok != nullptr) last_tok[b] = (n > 0) ? h[n - 1] : 0;
  }
  for (int i = tid; i < k; i += kThreads) draft[(size_t)b * k + i] = (i < len) ? h[start + i] : -1;
  if (stamp != nullptr) {
    __syncthreads();
    if (tid == 0) cs_stamp_end(stamp);
  }
}

}  // namespace

cs_status cs_launch_find_match(const int32_t* hist, const int32_t* hist_len, int B, int stride,
                               int gamma, int k, int policy, int32_t* match_pos, int32_t* draft,
                               int32_t* draft_len, int32_t* last_tok, const int32_t* skip,
                               cudaStream_t st, unsigned long long* stamp) {
  // no entry point reaches the kernel with a key longer than its compare loop or an unknown policy
  if (gamma < 1 || gamma > CS_MAX_GAMMA || (policy != CS_MATCH_LATEST && policy != CS_MATCH_FIRST) || k < 0 || B < 0)
    return CS_ERR_ARG;
  if (B == 0) return CS_OK;
  // 4096 candidates per CTA keep every thread at >= 4 vector iterations on long
  // histories; short ones use a single CTA per sequence
  int cl = 1;
  while (cl < 8 && stride > cl * 4096) cl *= 2;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(cl, B, 1);
  lc.blockDim = dim3(kThreads, 1, 1);
  lc.dynamicSmemBytes = 0;
  lc.stream = st;
  cudaLaunchAttribute at[2];
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cl;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  lc.attrs = at;
  // Launched as an ordinary stream-ordered kernel (cluster attribute only): the search opens
  // a decode step and reads the history the previous step's commit has just written, so the
  // step boundary is a full serialisation point.  (With the programmatic-launch attribute on
  // this cluster kernel the loop was observed to read a stale history.)
  lc.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&lc, k_find_match, (const int*)hist, (const int*)hist_len,
                                     stride, gamma, k, policy, (int*)match_pos, (int*)draft,
                                     (int*)draft_len, (int*)last_tok, (const int*)skip, stamp);
  return e == cudaSuccess ? CS_OK : CS_ERR_CUDA;
}
