// sdms_get_beams: several drafts per path.  One CTA per query path works out the B best paths of the
// pool of the last build (beam_dev.cuh) over node tables that it reserves in the workspace's table
// area and leaves empty again.
#include "sdms_internal.h"
#include "beam_dev.cuh"

namespace sdms {

namespace {

__global__ void __launch_bounds__(kWideThreads, 1) beam_kernel(Dev s, int B, int32_t* __restrict__ beam_tok,
                                                               int32_t* __restrict__ beam_len,
                                                               float* __restrict__ beam_value) {
  __shared__ long long sh_first;
  const int i = blockIdx.x, tid = threadIdx.x, D = s.D;
  int32_t* const my_tok = beam_tok + (size_t)i * B * D;
  const int M = s.q_mode[i] == Q_NONE ? 0 : min(s.q_cursor[i], s.q_reserved[i]);
  const int lcap = beam_lcap(M);
  if (tid == 0) {
    long long first = -1;
    if (M > 0 && M <= kWideMaxMatches) {
      const unsigned long long need = (unsigned long long)D << lcap;
      const unsigned long long at = atomicAdd(s.b_ctl, need);
      if (at + need <= s.w_slots) first = (long long)at;
      else atomicOr(s.status, SDMS_STATUS_TABLES_FULL);
    } else if (M > 0) {
      atomicOr(s.status, SDMS_STATUS_TABLES_FULL);
    }
    sh_first = first;
  }
  __syncthreads();
  if (sh_first < 0) {                                  // no match, or no room: no beam
    for (int x = tid; x < B * D; x += blockDim.x) my_tok[x] = -1;
    if (tid < B) { beam_len[(size_t)i * B + tid] = 0; beam_value[(size_t)i * B + tid] = 0.0f; }
    return;
  }
  beams_of_query(s, i, M, s.matches + s.q_off[i], (unsigned)sh_first, lcap, B, my_tok, beam_len + (size_t)i * B,
                 beam_value + (size_t)i * B);
}

// After a build with search mode 2: the paths that the build marked (more matches than its shared-memory
// search takes) get their best path here, in place of the greedy draft the build left them.
__global__ void __launch_bounds__(kWideThreads, 1) best_path_fix_kernel(Dev s, int32_t* __restrict__ draft_tok,
                                                                        int32_t* __restrict__ draft_len,
                                                                        float* __restrict__ draft_score,
                                                                        float* __restrict__ draft_edge_w) {
  grid_wait();
  grid_release();
  __shared__ long long sh_first;
  __shared__ float sh_value;
  const int i = blockIdx.x, tid = threadIdx.x, D = s.D;
  if (!s.bp_todo[i]) return;
  __syncthreads();
  if (tid == 0) s.bp_todo[i] = 0;
  const int M = min(s.q_cursor[i], s.q_reserved[i]);
  const int lcap = beam_lcap(M);
  if (tid == 0) {
    long long first = -1;
    if (M > 0 && M <= kWideMaxMatches) {
      const unsigned long long need = (unsigned long long)D << lcap;
      const unsigned long long at = atomicAdd(s.b_ctl + 1, need);
      if (at + need <= s.w_slots) first = (long long)at;
    }
    if (first < 0) atomicOr(s.status, SDMS_STATUS_SEARCH_FALLBACK);       // the greedy draft stays
    sh_first = first;
  }
  __syncthreads();
  if (sh_first < 0) return;
  beams_of_query(s, i, M, s.matches + s.q_off[i], (unsigned)sh_first, lcap, 1, draft_tok + (size_t)i * D, draft_len + i,
                 &sh_value, true, draft_score ? draft_score + (size_t)i * D : nullptr,
                 draft_edge_w ? draft_edge_w + (size_t)i * D : nullptr);
}

}  // namespace

cudaError_t launch_best_path_fix(const Dev& s, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                                 float* draft_edge_w, cudaStream_t stream) {
  cudaError_t e = cudaMemsetAsync(s.b_ctl + 1, 0, 8, stream);
  if (e != cudaSuccess) return e;
  return launch_overlapped(best_path_fix_kernel, dim3(s.P), dim3(kWideThreads), 0, stream, s, draft_tok, draft_len,
                           draft_score, draft_edge_w);
}

cudaError_t launch_beams(const Dev& s, int B, int32_t* beam_tok, int32_t* beam_len, float* beam_value,
                         cudaStream_t stream) {
  cudaError_t e = cudaMemsetAsync(s.b_ctl, 0, 8, stream);
  if (e != cudaSuccess) return e;
  beam_kernel<<<s.P, kWideThreads, 0, stream>>>(s, B, beam_tok, beam_len, beam_value);
  return cudaGetLastError();
}

}  // namespace sdms
