// State update and acceptance kernels.
//
// append_kernel : one CTA per path; writes tokens and fixed-point probabilities
//                 into the path store and inserts the n-grams (n = 1..k_max) that
//                 end at each new position into the prompt's hash tables.
// accept_kernel : one CTA per path; longest accepted prefix of the draft
//                 ("Draft acceptance"), optionally followed by the same append.
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

}  // namespace

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
