// Suffix matching for callers that must not allocate: the only device memory it
// needs beyond its arguments (two counters per path) lives in a fixed array that
// is part of this library's image on every GPU that loads it.
#include <mutex>
#include "sdms.h"
#include <cuda_runtime.h>

namespace {

constexpr int kTile = 1024;
constexpr int kThreads = 256;
constexpr int kMaxDevices = 64;

// counts [SDMS_NOALLOC_MAX_PATHS] followed by cursors [SDMS_NOALLOC_MAX_PATHS]: 128 KiB,
// resident on each device from the moment the library is loaded until the process ends.
static __device__ __align__(256) int32_t g_noalloc_scratch[2 * SDMS_NOALLOC_MAX_PATHS];

std::mutex g_mu;
int32_t* g_scratch_of_device[kMaxDevices] = {};

// The array's name is only a handle on the host; its address on the current
// device has to be asked for, once per device.
int scratch_on_current_device(int32_t** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SDMS_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_of_device[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return SDMS_ERR_CUDA;
    g_scratch_of_device[dev] = static_cast<int32_t*>(p);
  }
  *out = g_scratch_of_device[dev];
  return SDMS_OK;
}

__global__ void noalloc_clear_kernel(int32_t* scratch, int P) {
  const int x = blockIdx.x * blockDim.x + threadIdx.x;
  if (x < P) { scratch[x] = 0; scratch[SDMS_NOALLOC_MAX_PATHS + x] = 0; }
}

// One CTA per 1024-token tile of one path j; every other path of the prompt that
// has a query compares its last k tokens against each window of the tile.
template <bool FILL>
__global__ void __launch_bounds__(kThreads) noalloc_scan_kernel(
    const int32_t* __restrict__ tok, const int32_t* __restrict__ len, int N, int L, int k, int tiles,
    int32_t* scratch, const int32_t* __restrict__ offsets, int32_t* __restrict__ gpos, size_t cap) {
  const int j = blockIdx.x / tiles;
  const int t0 = (blockIdx.x % tiles) * kTile;
  const int len_j = len[j];
  const int e_lo = max(t0, k - 1), e_hi = min(t0 + kTile - 1, len_j - 2);
  if (e_lo > e_hi) return;
  __shared__ int32_t sh[SDMS_MAX_K + kTile];
  const int32_t* row = tok + (size_t)j * L;
  for (int x = threadIdx.x; x < SDMS_MAX_K + kTile; x += blockDim.x) {
    const int idx = t0 - SDMS_MAX_K + x;
    sh[x] = (idx >= 0 && idx < L) ? row[idx] : -1;
  }
  __syncthreads();
  int32_t* counts = scratch;
  int32_t* cursors = scratch + SDMS_NOALLOC_MAX_PATHS;
  const int g = j / N;
  for (int i = g * N; i < (g + 1) * N; ++i) {
    const int len_i = len[i];
    if (i == j || len_i < k || len_i >= L) continue;
    const int32_t* q = tok + (size_t)i * L + (len_i - k);
    int found = 0;
    for (int e = e_lo + threadIdx.x; e <= e_hi; e += blockDim.x) {
      const int32_t* w = sh + SDMS_MAX_K + (e - t0) - (k - 1);
      bool same = true;
      for (int t = 0; t < k; ++t) same = same && (w[t] == q[t]);
      if (!same) continue;
      if (FILL) {
        const size_t at = (size_t)offsets[i] + (size_t)atomicAdd(&cursors[i], 1);
        if (at < cap) gpos[at] = j * L + e;
      } else {
        ++found;
      }
    }
    if (!FILL) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) found += __shfl_xor_sync(0xffffffffu, found, o);
      if ((threadIdx.x & 31) == 0 && found) atomicAdd(&counts[i], found);
    }
  }
}

__global__ void __launch_bounds__(1024) noalloc_offsets_kernel(const int32_t* scratch, int P, int32_t* offsets) {
  __shared__ int warp_tot[32];
  __shared__ int carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (int base = 0; base < P; base += blockDim.x) {
    const int i = base + threadIdx.x;
    const int v = i < P ? scratch[i] : 0;
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
    if (lane == 31) warp_tot[wid] = x;
    __syncthreads();
    if (wid == 0) {
      int w = warp_tot[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, w, o); if (lane >= o) w += y; }
      warp_tot[lane] = w;
    }
    __syncthreads();
    if (i < P) offsets[i] = carry + (wid ? warp_tot[wid - 1] : 0) + x - v;
    __syncthreads();
    if (threadIdx.x == 0) carry += warp_tot[31];
    __syncthreads();
  }
  if (threadIdx.x == 0) offsets[P] = carry;
}

}  // namespace

extern "C" int sdms_match_noalloc(const int32_t* d_tok, const int32_t* d_len, int32_t num_groups,
                                  int32_t paths_per_group, int32_t capacity, int32_t k, int32_t* d_offsets,
                                  int32_t* d_gpos, size_t cap, void* stream) {
  if (!d_tok || !d_len || !d_offsets || (!d_gpos && cap)) return SDMS_ERR_INVALID_ARG;
  if (num_groups < 1 || paths_per_group < 1 || capacity < 2 || k < 1 || k > SDMS_MAX_K) return SDMS_ERR_INVALID_ARG;
  if (paths_per_group > SDMS_MAX_PATHS_PER_GROUP) return SDMS_ERR_INVALID_ARG;
  const long long P = (long long)num_groups * paths_per_group;
  if (P > SDMS_NOALLOC_MAX_PATHS) return SDMS_ERR_TOO_LARGE;          // the fixed scratch holds no more
  if (P * capacity > 0x7fffffffLL) return SDMS_ERR_INVALID_ARG;
  // offsets are int32: even if every position matched every query of its prompt the total must fit
  if (P * paths_per_group * capacity > 0x7fffffffLL) return SDMS_ERR_TOO_LARGE;
  int32_t* scratch = nullptr;
  const int rc = scratch_on_current_device(&scratch);
  if (rc != SDMS_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const int tiles = (capacity + kTile - 1) / kTile;
  const unsigned grid = (unsigned)(P * tiles);
  // the array still holds the previous call's counters: start from zero
  noalloc_clear_kernel<<<((int)P + 255) / 256, 256, 0, st>>>(scratch, (int)P);
  noalloc_scan_kernel<false><<<grid, kThreads, 0, st>>>(d_tok, d_len, paths_per_group, capacity, k, tiles, scratch,
                                                        nullptr, nullptr, 0);
  noalloc_offsets_kernel<<<1, 1024, 0, st>>>(scratch, (int)P, d_offsets);
  noalloc_scan_kernel<true><<<grid, kThreads, 0, st>>>(d_tok, d_len, paths_per_group, capacity, k, tiles, scratch,
                                                       d_offsets, d_gpos, cap);
  return cudaGetLastError() == cudaSuccess ? SDMS_OK : SDMS_ERR_CUDA;
}
