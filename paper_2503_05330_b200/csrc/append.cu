// State update and acceptance kernels.
//
// append_kernel : one CTA per path; writes tokens and fixed-point probabilities
//                 into the path store and inserts the n-grams (n = 1..k_max) that
//                 end at each new position into the prompt's hash tables.
// accept_kernel : one CTA per path; longest accepted prefix of the draft
//                 ("Draft acceptance"), optionally followed by the same append.
// trim_*        : sliding window: shift the histories, empty and refill the tables.
#include "sdms_internal.h"
#include "append_dev.cuh"

namespace sdms {

namespace {

__global__ void __launch_bounds__(128) append_kernel(Dev s, const int32_t* __restrict__ tokens,
                                                     const float* __restrict__ logprobs,
                                                     const int32_t* __restrict__ counts, int row_width) {
  grid_wait();
  grid_release();
  const int p = blockIdx.x;
  __shared__ int sh_len0, sh_n, sh_bad;
  __shared__ uint32_t sh_st;
  __shared__ int32_t sh_rec[kRecWords];
  if (threadIdx.x < kRecWords) sh_rec[threadIdx.x] = s.rec[(size_t)p * kRecWords + threadIdx.x];
  if (threadIdx.x == 0) {
    uint32_t st = 0;
    int n = counts[p];
    if (n < 0) { st |= SDMS_STATUS_BAD_COUNT; n = 0; }
    if (n > row_width) { st |= SDMS_STATUS_BAD_COUNT; n = row_width; }
    const int len0 = sh_rec[0];
    if (n > s.L - len0) { st |= SDMS_STATUS_CAPACITY; n = s.L - len0; }
    sh_len0 = len0; sh_n = n; sh_bad = n; sh_st = st;
  }
  __syncthreads();
  const int32_t* in_tok = tokens + (size_t)p * row_width;
  const float* in_lp = logprobs + (size_t)p * row_width;
  for (int a = threadIdx.x; a < sh_n; a += blockDim.x) {
    const int32_t t = in_tok[a];
    if (t < 0 || t >= s.V) atomicMin(&sh_bad, a);
  }
  __syncthreads();
  uint32_t st = 0;
  const int n = sh_bad;
  if (threadIdx.x == 0 && n < sh_n) st |= SDMS_STATUS_BAD_TOKEN;
  append_tokens(s, p, sh_len0, n, in_tok, in_lp, sh_rec, &st);
  if (st) atomicOr(&sh_st, st);
  __syncthreads();
  if (threadIdx.x == 0 && sh_st) atomicOr(s.status, sh_st);
}

__global__ void __launch_bounds__(128) accept_kernel(Dev s, const int32_t* __restrict__ draft_tok,
                                                     const int32_t* __restrict__ draft_len,
                                                     const int32_t* __restrict__ sampled,
                                                     const float* __restrict__ sampled_lp,
                                                     int32_t* __restrict__ accept_len) {
  grid_wait();
  grid_release();
  accept_commit_phase(s, blockIdx.x, draft_tok, draft_len, sampled, sampled_lp, accept_len);
}

// sdms_trim, first launch: path p keeps its newest keep[p] tokens, moved to the front of its store.
__global__ void __launch_bounds__(128) trim_shift_kernel(Dev s, const int32_t* __restrict__ keep) {
  grid_wait();
  grid_release();
  const int p = blockIdx.x;
  const int len = s.len[p], want = keep[p];
  if (want < 0) {
    if (threadIdx.x == 0) atomicOr(s.status, SDMS_STATUS_BAD_COUNT);
    return;
  }
  if (want >= len) return;
  const int shift = len - want;
  int32_t* tok = s.tok + (size_t)p * s.L;
  int32_t* pq = s.pq + (size_t)p * s.L;
  // a block of the kept tokens is read whole before any of it is written: the source of a later
  // block lies behind everything written so far
  for (int base = 0; base < want; base += blockDim.x) {
    const int x = base + threadIdx.x;
    int32_t t = 0, q = 0;
    if (x < want) { t = tok[x + shift]; q = pq[x + shift]; }
    __syncthreads();
    if (x < want) { tok[x] = t; pq[x] = q; }
    __syncthreads();
  }
  int32_t* rec = s.rec + (size_t)p * kRecWords;
  if (threadIdx.x == 0) { s.len[p] = want; rec[0] = want; s.g_trim[p / s.N] = 1; }
  if (threadIdx.x >= 1 && threadIdx.x < kRecWords && (int)threadIdx.x > want) rec[threadIdx.x] = 0;   // tokens that are gone
}

// Second launch: the tables of the prompts that changed become empty.
__global__ void __launch_bounds__(256) trim_clear_kernel(Dev s) {
  grid_wait();
  grid_release();
  const size_t per_group = (size_t)s.idx_n * s.table_cap * kBucketWords / 4;      // 16-byte words of a prompt's tables
  uint4* index = reinterpret_cast<uint4*>(s.index);
  for (size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x; x < per_group * s.G; x += (size_t)gridDim.x * blockDim.x)
    if (s.g_trim[x / per_group]) index[x] = make_uint4(0u, 0u, 0u, 0u);
}

// Third launch: every n-gram (n = 1..k_max) of every path of those prompts goes into the tables again.
__global__ void __launch_bounds__(128) trim_reindex_kernel(Dev s) {
  grid_wait();
  grid_release();
  const int p = blockIdx.x, g = p / s.N;
  if (!s.g_trim[g]) return;
  const int len = s.len[p];
  const int32_t* tok = s.tok + (size_t)p * s.L;
  const uint32_t lbase = (uint32_t)(p - g * s.N) * (uint32_t)s.L;
  uint32_t st = 0;
  for (int w = threadIdx.x; w < len * s.idx_n; w += blockDim.x) {
    const int pos = w / s.idx_n, nn = w % s.idx_n + 1;
    if (pos + 1 < nn) continue;
    uint64_t h = gram_init(nn);
    for (int t = pos - nn + 1; t <= pos; ++t) h = gram_step(h, tok[t]);
    index_insert(s, g, nn, gram_final(h), lbase + (uint32_t)pos, &st);
  }
  if (st) atomicOr(s.status, st);
}

}  // namespace

cudaError_t launch_trim(const Dev& s, int phase, const int32_t* keep, cudaStream_t stream) {
  if (phase == 0) return launch_overlapped(trim_shift_kernel, dim3(s.P), dim3(128), 0, stream, s, keep);
  if (phase == 1) return launch_overlapped(trim_clear_kernel, dim3(148 * 8), dim3(256), 0, stream, s);
  return launch_overlapped(trim_reindex_kernel, dim3(s.P), dim3(128), 0, stream, s);
}

cudaError_t launch_append(const Dev& s, const int32_t* tokens, const float* logprobs, const int32_t* counts,
                          int row_width, cudaStream_t stream) {
  return launch_overlapped(append_kernel, dim3(s.P), dim3(128), 0, stream, s, tokens, logprobs, counts, row_width);
}

cudaError_t launch_accept(const Dev& s, const int32_t* draft_tok, const int32_t* draft_len,
                          const int32_t* sampled, const float* sampled_lp, int32_t* accept_len,
                          cudaStream_t stream) {
  return launch_overlapped(accept_kernel, dim3(s.P), dim3(128), 0, stream, s, draft_tok, draft_len, sampled, sampled_lp,
                           accept_len);
}

}  // namespace sdms
