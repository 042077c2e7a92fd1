// Host-side launchers, one per translation unit of kernels.
#pragma once
#include "sdms_dev.cuh"

namespace sdms {

// Launch with programmatic stream serialization: the kernel's CTAs may be scheduled before the
// previous kernel on the stream has finished; the kernel itself waits (grid_wait) before it reads
// or writes anything.
template <class... KArgs, class... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

cudaError_t launch_append(const Dev& s, const int32_t* tokens, const float* logprobs, const int32_t* counts,
                          int row_width, cudaStream_t stream);
cudaError_t launch_accept(const Dev& s, const int32_t* draft_tok, const int32_t* draft_len,
                          const int32_t* sampled, const float* sampled_lp, int32_t* accept_len,
                          cudaStream_t stream);
cudaError_t launch_probe(const Dev& s, int k, int skip_done, cudaStream_t stream);
cudaError_t launch_scan(const Dev& s, int k, cudaStream_t stream);
// tolerance 1 on large prompts: mark the queries, count, hand out slices, fill (four launches)
cudaError_t launch_fuzzy_match(const Dev& s, int k, int skip_done, cudaStream_t stream);
// round: 0 for an ordinary build; kRound* flags, k and used_k for one round of a back-off build on a large prompt
cudaError_t launch_dag(const Dev& s, bool with_export, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                       float* draft_edge_w, cudaStream_t stream, int round = 0, int k = 0, int32_t* used_k = nullptr);
cudaError_t launch_build_fused(const Dev& s, int k_hi, int k_lo, int32_t* draft_tok, int32_t* draft_len,
                               float* draft_score, float* draft_edge_w, int32_t* used_k, cudaStream_t stream);
// phase 0: shift the histories; 1: empty the index tables of the prompts that changed; 2: index them again
cudaError_t launch_trim(const Dev& s, int phase, const int32_t* keep, cudaStream_t stream);
bool step_kernel_fits(const Dev& s);
int build_cluster_size(const Dev& s);
cudaError_t launch_step(const Dev& s, int k, int k_lo, const int32_t* sampled, const float* sampled_lp,
                        int32_t* accept_len, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                        float* draft_edge_w, int32_t* used_k, cudaStream_t stream);
cudaError_t launch_compact_matches(const Dev& s, int32_t* offsets, int32_t* gpos, size_t cap, cudaStream_t stream);
// queries with many matches, aggregated by all SMs (dag_wide.cu)
int wide_kernel_grid();
cudaError_t launch_wait_timeout(const Dev& s, long long cycles, cudaStream_t stream);
cudaError_t launch_dag_wide(const Dev& s, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                            float* draft_edge_w, cudaStream_t stream);
cudaError_t launch_beams(const Dev& s, int B, int32_t* beam_tok, int32_t* beam_len, float* beam_value,
                         cudaStream_t stream);
cudaError_t launch_best_path_fix(const Dev& s, int32_t* draft_tok, int32_t* draft_len, float* draft_score,
                                 float* draft_edge_w, cudaStream_t stream);
cudaError_t dag_kernel_setup();
cudaError_t scan_kernel_setup();

}  // namespace sdms
