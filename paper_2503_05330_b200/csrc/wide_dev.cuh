// Hand-over of a query with many matches to the device-wide aggregation pass (dag_wide.cu).
#pragma once
#include "sdms_dev.cuh"

namespace sdms {

// log2 of the slots of one layer's node table: a power of two above 5/4 of the matches, so that a
// layer in which every candidate is a node of its own still leaves a fifth of the slots free.
__device__ __forceinline__ int wide_lcap(int M) {
  int l = 6;
  while ((1ll << l) < (long long)M + (M >> 2) + 1) ++l;
  return l;
}

// Called by every thread of the query's CTA.  Reserves table slots for all D layers and enters the
// query in the list the wide pass works through; false (for all threads) if the pass is not in use,
// the list is full or the slots have run out - the caller then aggregates the query itself.
__device__ __forceinline__ bool wide_register(const Dev& s, int i, int M) {
  __shared__ int sh_wide_q;
  if (s.w_slots == 0 || M > kWideMaxMatches) return false;
  if (threadIdx.x == 0) {
    int q = -1;
    const int lcap = wide_lcap(M);
    const unsigned long long need = (unsigned long long)s.D << lcap;
    const unsigned long long first = atomicAdd(&s.w_ctl[1], need);
    if (first + need <= s.w_slots) {
      const unsigned long long n = atomicAdd(&s.w_ctl[0], 1ull);
      if (n < (unsigned long long)kMaxWide) {
        q = (int)n;
        s.w_desc[q] = make_int4(i, M, lcap, (int)(unsigned)first);
        atomicMax(&s.w_ctl[3], first + need);
      }
    }
    sh_wide_q = q;
  }
  __syncthreads();
  const int q = sh_wide_q;
  if (q >= 0 && threadIdx.x < SDMS_MAX_DRAFT) {
    s.w_pred[(size_t)q * SDMS_MAX_DRAFT + threadIdx.x] = WidePred{0ull, 0ull};
    s.w_edge[(size_t)q * SDMS_MAX_DRAFT + threadIdx.x] = 0ull;
  }
  return q >= 0;
}

}  // namespace sdms
