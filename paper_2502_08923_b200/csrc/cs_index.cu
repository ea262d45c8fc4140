// Device-resident index of all gamma-grams of the accepted sequences (Sec. 3.1: the paper keeps
// a hash map from every gamma-token subsequence to where it occurs, O(gamma) work per appended
// token and per lookup).  cs_find_match scans the history instead, which is cheaper up to a few
// tens of thousands of tokens; this index makes the search independent of the history length.
//
// One open-addressing table per sequence.  A slot holds the first and the latest start
// position of one gamma-gram; the gram itself is not stored - it is read back from the history
// at the slot's first position, so a lookup compares tokens, never just hashes, and the result
// is exactly the scan's.  The non-overlap rule (a match must end before the key starts,
// p0 <= n - 2*gamma; App. B.3 step 1(c)) is kept by inserting late: an update at history
// length n only inserts starts p <= n - 2*gamma, so whatever a lookup finds is admissible and
// "latest" is simply the latest start inserted.  A lookup therefore belongs to the history
// length of the last update.  Probing is linear and bounded by the table size.
#include "cs_common.cuh"

namespace {

constexpr int kIdxThreads = 256;

__host__ __device__ inline unsigned idx_slots(int capacity_tokens) {
  unsigned s = 64;
  while (s < 2u * (unsigned)capacity_tokens) s <<= 1;
  return s;
}

__device__ __forceinline__ unsigned gram_hash(const int* g, int gamma) {
  unsigned long long h = 0x9E3779B97F4A7C15ull;
  for (int j = 0; j < gamma; ++j) {
    h ^= (unsigned long long)(unsigned)g[j];
    h *= 0xBF58476D1CE4E5B9ull;
    h ^= h >> 29;
  }
  return (unsigned)(h ^ (h >> 32));
}

__device__ __forceinline__ bool gram_equal(const int* a, const int* b, int gamma) {
  bool eq = true;
  for (int j = 0; j < gamma; ++j) eq = eq && (a[j] == b[j]);
  return eq;
}

// Insert every start p in [indexed_len[b], hist_len[b] - 2*gamma] of every sequence.
__global__ void k_gram_insert(int2* __restrict__ table, unsigned slots, const int* __restrict__ hist,
                              const int* __restrict__ hist_len, int stride, int gamma,
                              const int* __restrict__ indexed_len, int* __restrict__ status) {
  const int b = blockIdx.y;
  const int* h = hist + (size_t)b * stride;
  int2* T = table + (size_t)b * slots;
  int n = hist_len[b];
  n = n > stride ? stride : n;
  const int lo = max(0, indexed_len[b]), hi = n - 2 * gamma;
  for (int p = lo + blockIdx.x * blockDim.x + threadIdx.x; p <= hi; p += gridDim.x * blockDim.x) {
    unsigned s = gram_hash(h + p, gamma) & (slots - 1);
    bool placed = false;
    for (unsigned probe = 0; probe < slots && !placed; ++probe, s = (s + 1) & (slots - 1)) {
      int first = atomicCAS(&T[s].x, -1, p);        // claim an empty slot for this gram
      if (first == -1) first = p;
      if (gram_equal(h + first, h + p, gamma)) {
        atomicMin(&T[s].x, p);
        atomicMax(&T[s].y, p);
        placed = true;
      }
    }
    if (!placed) atomicOr(status, CS_DEV_CAPACITY);   // table full: more tokens than it was sized for
  }
}

__global__ void k_gram_commit(const int* __restrict__ hist_len, int stride, int gamma, int B, int* indexed_len) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int n = hist_len[b];
  n = n > stride ? stride : n;
  indexed_len[b] = max(max(0, indexed_len[b]), n - 2 * gamma + 1);
}

// Look the last gamma tokens up and gather the draft (same outputs as the scan).
__global__ void k_gram_lookup(const int2* __restrict__ table, unsigned slots, const int* __restrict__ hist,
                              const int* __restrict__ hist_len, int stride, int gamma, int k, int policy,
                              int* __restrict__ match_pos, int* __restrict__ draft, int* __restrict__ draft_len,
                              int* __restrict__ last_tok, const int* __restrict__ skip) {
  const int b = blockIdx.x;
  const int* h = hist + (size_t)b * stride;
  const int2* T = table + (size_t)b * slots;
  int n = hist_len[b];
  n = n > stride ? stride : (n < 0 ? 0 : n);
  const bool dead = (skip != nullptr && skip[b] != 0);   // a finished sequence of the loop: no match, no draft
  __shared__ int s_p0;
  if (threadIdx.x == 0) {
    int p0 = -1;
    if (n >= 2 * gamma && !dead) {
      const int* key = h + n - gamma;
      unsigned s = gram_hash(key, gamma) & (slots - 1);
      for (unsigned probe = 0; probe < slots; ++probe, s = (s + 1) & (slots - 1)) {
        const int2 e = T[s];
        if (e.x < 0) break;                            // empty slot: the gram was never inserted
        if (gram_equal(h + e.x, key, gamma)) {
          p0 = (policy == CS_MATCH_LATEST) ? e.y : e.x;
          break;
        }
      }
    }
    s_p0 = p0;
  }
  __syncthreads();
  const int p0 = s_p0, start = p0 + gamma;
  const int len = (p0 < 0) ? 0 : min(k, n - start);
  if (threadIdx.x == 0) {
    match_pos[b] = p0;
    draft_len[b] = len;
    if (last_tok != nullptr) last_tok[b] = (n > 0) ? h[n - 1] : 0;
  }
  for (int i = threadIdx.x; i < k; i += blockDim.x) draft[(size_t)b * k + i] = (i < len) ? h[start + i] : -1;
}

}  // namespace

// The loop's use of the index (App. B.3 step 1 by lookup, step 2(d) by insertion): same outputs as
// the scan's launcher; table overflow goes to `status` (the context's status word).
cs_status cs_launch_gram_lookup(const void* index, int B, int capacity_tokens, const int32_t* hist, const int32_t* hist_len,
                                int stride, int gamma, int k, int policy, int32_t* match_pos, int32_t* draft,
                                int32_t* draft_len, int32_t* last_tok, const int32_t* skip, cudaStream_t st) {
  if (gamma < 1 || gamma > CS_MAX_GAMMA || (policy != CS_MATCH_LATEST && policy != CS_MATCH_FIRST) || k < 0 || B < 1)
    return CS_ERR_ARG;
  k_gram_lookup<<<B, 128, 0, st>>>(static_cast<const int2*>(index), idx_slots(capacity_tokens), hist, hist_len, stride, gamma, k,
                                   policy, match_pos, draft, draft_len, last_tok, skip);
  return cudaGetLastError() == cudaSuccess ? CS_OK : CS_ERR_CUDA;
}

cs_status cs_launch_gram_update(void* index, int B, int capacity_tokens, const int32_t* hist, const int32_t* hist_len,
                                int stride, int gamma, int max_chunks, int* status, cudaStream_t st) {
  const unsigned slots = idx_slots(capacity_tokens);
  int* ilen = reinterpret_cast<int*>(static_cast<char*>(index) + (size_t)B * slots * sizeof(int2));
  int chunks = cs_ceil_div(stride, kIdxThreads);
  chunks = chunks < 1 ? 1 : (chunks > max_chunks ? max_chunks : chunks);
  k_gram_insert<<<dim3(chunks, B), kIdxThreads, 0, st>>>(static_cast<int2*>(index), slots, hist, hist_len, stride, gamma, ilen,
                                                        status != nullptr ? status : ilen + B);
  k_gram_commit<<<cs_ceil_div(B, 128), 128, 0, st>>>(hist_len, stride, gamma, B, ilen);
  return cudaGetLastError() == cudaSuccess ? CS_OK : CS_ERR_CUDA;
}

extern "C" size_t cs_gram_index_bytes(int B, int capacity_tokens) {
  if (B < 1 || capacity_tokens < 1) return 0;
  return (size_t)B * idx_slots(capacity_tokens) * sizeof(int2) + (size_t)B * sizeof(int) + 256;
}

// layout of the caller's buffer: [B][slots] int2, then indexed_len [B], then the status word
static int* idx_len_ptr(void* index, int B, int capacity_tokens) {
  return reinterpret_cast<int*>(static_cast<char*>(index) + (size_t)B * idx_slots(capacity_tokens) * sizeof(int2));
}

extern "C" cs_status cs_gram_index_reset(void* index, int B, int capacity_tokens, void* stream) {
  if (index == nullptr || B < 1 || capacity_tokens < 1) return CS_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t tbl = (size_t)B * idx_slots(capacity_tokens) * sizeof(int2);
  if (cudaMemsetAsync(index, 0xFF, tbl, st) != cudaSuccess) return CS_ERR_CUDA;                           // every slot (-1, -1)
  if (cudaMemsetAsync(static_cast<char*>(index) + tbl, 0, (size_t)B * sizeof(int) + 256, st) != cudaSuccess) return CS_ERR_CUDA;
  return CS_OK;
}

extern "C" cs_status cs_gram_index_update(void* index, int B, int capacity_tokens, const int32_t* hist,
                                          const int32_t* hist_len, int stride, int gamma, void* stream) {
  if (index == nullptr || hist == nullptr || hist_len == nullptr || B < 1 || B > 65535 || capacity_tokens < 1 || stride < 0)
    return CS_ERR_ARG;
  if (gamma < 1 || gamma > CS_MAX_GAMMA) return CS_ERR_ARG;
  return cs_launch_gram_update(index, B, capacity_tokens, hist, hist_len, stride, gamma, 64, nullptr,
                               static_cast<cudaStream_t>(stream));
}

extern "C" cs_status cs_find_match_indexed(const void* index, int B, int capacity_tokens, const int32_t* hist,
                                           const int32_t* hist_len, int stride, int gamma, int k, cs_match_policy policy,
                                           int32_t* match_pos, int32_t* draft, int32_t* draft_len, void* stream) {
  if (index == nullptr || hist == nullptr || hist_len == nullptr || match_pos == nullptr || draft_len == nullptr ||
      (draft == nullptr && k > 0) || B < 1 || k < 0 || stride < 0 || capacity_tokens < 1)
    return CS_ERR_ARG;
  if (gamma < 1 || gamma > CS_MAX_GAMMA) return CS_ERR_ARG;
  if (policy != CS_MATCH_LATEST && policy != CS_MATCH_FIRST) return CS_ERR_ARG;
  return cs_launch_gram_lookup(index, B, capacity_tokens, hist, hist_len, stride, gamma, k, (int)policy, match_pos, draft,
                               draft_len, nullptr, nullptr, static_cast<cudaStream_t>(stream));
}

// 0 if every insertion so far found a slot, CS_ERR_CAPACITY otherwise; synchronises the stream.
extern "C" cs_status cs_gram_index_status(const void* index, int B, int capacity_tokens, void* stream) {
  if (index == nullptr || B < 1 || capacity_tokens < 1) return CS_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int bits = 0;
  const int* status = idx_len_ptr(const_cast<void*>(index), B, capacity_tokens) + B;
  if (cudaMemcpyAsync(&bits, status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return CS_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return CS_ERR_CUDA;
  return (bits & CS_DEV_CAPACITY) ? CS_ERR_CAPACITY : CS_OK;
}
