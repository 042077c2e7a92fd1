// Fuzzy suffix matching (Eq. 4, tolerance 1) on prompts too large for the single-launch build.
//
// A position (j, e) matches query path i when some window of k - 1, k or k + 1 tokens that ends at e is
// within edit distance 1 of the query; each position counts once.  Index counts say nothing about how
// many such positions there are, so the match slices are sized by counting first:
//   fuzzy_prepare  every path with a query (k tokens, not full) is marked for scanning, counters zeroed
//   fuzzy_scan     (count) one CTA per 1024-token tile of one path j: positions that can end a match of
//                  ANY query of the prompt are picked out by a bit table, then tested against every query
//   fuzzy_alloc    slices handed out from the match list by the counts
//   fuzzy_scan     (fill) the same scan writes the positions
// after which dag_kernel (and the wide pass) aggregate as for exact matching.
//
// The filter.  Let q be the query, |q| = k >= 2.  A window within one edit of q that ends at e either ends
// in q's last token, or differs from q only at its end: then the token at e or the one before it is
// q[k-1] or q[k-2] (substitution of the last token: tok[e-1] = q[k-2]; last token deleted: tok[e] =
// q[k-2]; a token appended: tok[e-1] = q[k-1]).  So a position passes when tok[e] or tok[e-1] hashes to
// a bit that some query set for q[k-1] or q[k-2].  With k = 1 every position is within one substitution
// of every query and nothing is filtered.
//
// The test.  With a = common prefix and b = common suffix of q and a window s' (each at most the shorter
// length), the edit distance is at most 1 iff a + b >= max(|q|, |s'|) - 1.
#include "sdms_internal.h"

namespace sdms {

namespace {

constexpr int kFzTile = 1024;
constexpr int kFzThreads = 256;
constexpr int kFzHalo = SDMS_MAX_K + 1;            // tokens in front of a tile that a window may reach
constexpr int kFzBits = 65536;
constexpr int kFzQueries = 128;                    // queries whose tokens are staged at a time

__device__ __forceinline__ uint32_t fz_bit(int32_t tok) { return ((uint32_t)tok * 2654435761u) >> 16; }

__global__ void __launch_bounds__(256) fuzzy_prepare_kernel(Dev s, int k, int skip_done) {
  grid_wait();
  grid_release();
  if (blockIdx.x == 0 && threadIdx.x < kWideCtlWords && s.w_grid) s.w_ctl[threadIdx.x] = 0ull;   // the wide pass of this build starts with an empty list
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= s.P) return;
  if (skip_done && s.q_mode[i] == Q_DONE) return;                // back-off: this path has its matches from a longer suffix
  const int len = s.len[i];
  s.q_fp[i] = 0u;
  s.q_mode[i] = len >= k && len < s.L ? Q_SCAN : Q_NONE;
  s.q_reserved[i] = 0; s.q_off[i] = 0; s.q_cursor[i] = 0;
}

__global__ void __launch_bounds__(256) fuzzy_alloc_kernel(Dev s) {
  grid_wait();
  grid_release();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= s.P || s.q_mode[i] != Q_SCAN) return;
  const long long count = s.q_reserved[i];
  const long long at = (long long)atomicAdd(s.match_cursor, (unsigned long long)count);
  if (at + count > s.match_cap) {
    s.q_mode[i] = Q_NONE; s.q_reserved[i] = 0;
    atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
  } else {
    s.q_off[i] = (int32_t)at;
  }
}

// Is some window that ends at position e of `row` (tokens row[0 .. e]) within one edit of q[0 .. k)?
__device__ __forceinline__ bool one_edit_end(const int32_t* row, int e, const int32_t* q, int k) {
  int b = 0;
  while (b < k && b <= e && row[e - b] == q[k - 1 - b]) ++b;
  for (int n = max(1, k - 1); n <= k + 1; ++n) {
    if (e - n + 1 < 0) break;
    const int shorter = min(k, n), need = max(k, n) - 1 - min(b, shorter);
    if (need <= 0) return true;
    if (need > shorter) continue;
    int a = 0;
    while (a < need && row[e - n + 1 + a] == q[a]) ++a;
    if (a >= need) return true;
  }
  return false;
}

template <bool FILL>
__global__ void __launch_bounds__(kFzThreads) fuzzy_scan_kernel(Dev s, int k, int tiles) {
  __shared__ int32_t sh_tok[kFzHalo + kFzTile];            // sh_tok[kFzHalo + x] = token at t0 + x
  __shared__ uint32_t sh_bits[kFzBits / 32];
  __shared__ int32_t sh_q[kFzQueries][SDMS_MAX_K];
  __shared__ int32_t sh_qi[kFzQueries];
  __shared__ int sh_cand[kFzTile];
  __shared__ int sh_ncand, sh_nq;
  const int tid = threadIdx.x;
  const int j = blockIdx.x / tiles, t0 = (blockIdx.x - j * tiles) * kFzTile;
  const int g = j / s.N, len_j = s.len[j];
  const int e_hi = min(t0 + kFzTile - 1, len_j - 2);        // last position of the tile with a follower
  if (t0 > e_hi) return;
  const int32_t* row = s.tok + (size_t)j * s.L;
  for (int x = tid; x < kFzHalo + kFzTile; x += blockDim.x) {
    const int at = t0 - kFzHalo + x;
    sh_tok[x] = at >= 0 && at < len_j ? row[at] : -1;
  }
  for (int x = tid; x < kFzBits / 32; x += blockDim.x) sh_bits[x] = 0u;
  if (tid == 0) sh_ncand = 0;
  // tokens and path lengths are older than the kernels this one follows (their CTAs let it start only after their own
  // wait): the tile was staged while those drained; the queries' state is read from here on
  grid_wait();
  grid_release();
  __syncthreads();
  // the tokens that can sit at the end of a match: the last two of every query of the prompt
  if (k >= 2)
    for (int n = tid; n < s.N; n += blockDim.x) {
      const int i = g * s.N + n;
      if (i == j || s.q_mode[i] != Q_SCAN) continue;
      const int32_t* rec = s.rec + (size_t)i * kRecWords;   // rec[1 + t] = token t places from the end
      const uint32_t b0 = fz_bit(rec[1]), b1 = fz_bit(rec[2]);
      atomicOr(&sh_bits[b0 >> 5], 1u << (b0 & 31));
      atomicOr(&sh_bits[b1 >> 5], 1u << (b1 & 31));
    }
  __syncthreads();
  for (int x = tid; x <= e_hi - t0; x += blockDim.x) {
    bool pass = k < 2;
    if (!pass) {
      const uint32_t b0 = fz_bit(sh_tok[kFzHalo + x]);
      pass = sh_bits[b0 >> 5] >> (b0 & 31) & 1u;
      if (!pass && t0 + x >= 1) {
        const uint32_t b1 = fz_bit(sh_tok[kFzHalo + x - 1]);
        pass = sh_bits[b1 >> 5] >> (b1 & 31) & 1u;
      }
    }
    if (pass) sh_cand[atomicAdd(&sh_ncand, 1)] = x;
  }
  __syncthreads();
  const int ncand = sh_ncand;
  if (ncand == 0) return;
  // the candidates against every query of the prompt, kFzQueries queries at a time
  for (int n0 = 0; n0 < s.N; n0 += kFzQueries) {
    __syncthreads();
    if (tid == 0) sh_nq = 0;
    __syncthreads();
    for (int n = n0 + tid; n < min(s.N, n0 + kFzQueries); n += blockDim.x) {
      const int i = g * s.N + n;
      if (i == j || s.q_mode[i] != Q_SCAN) continue;
      const int at = atomicAdd(&sh_nq, 1);
      sh_qi[at] = i;
      const int32_t* rec = s.rec + (size_t)i * kRecWords;
      for (int t = 0; t < k; ++t) sh_q[at][t] = rec[k - t];   // oldest token first
    }
    __syncthreads();
    const int nq = sh_nq;
    for (int x = tid; x < ncand * nq; x += blockDim.x) {
      const int c = x / nq, q = x - c * nq;
      const int pos = sh_cand[c];                              // position t0 + pos
      // the window may reach kFzHalo tokens in front of the tile; what lies before the path's start is -1
      const int reach = min(t0 + pos, kFzHalo + pos);          // tokens available before (and at) the position, minus one
      if (!one_edit_end(sh_tok + kFzHalo + pos - reach, reach, sh_q[q], k)) continue;
      const int i = sh_qi[q];
      if (FILL) {
        const int at = atomicAdd(&s.q_cursor[i], 1);
        if (at < s.q_reserved[i]) s.matches[(size_t)s.q_off[i] + at] = j * s.L + t0 + pos;
      } else {
        atomicAdd(&s.q_reserved[i], 1);
      }
    }
  }
}

}  // namespace

// probe + scan of a build with tolerance 1 on a context that does not take the single-launch build
cudaError_t launch_fuzzy_match(const Dev& s, int k, int skip_done, cudaStream_t stream) {
  const int tiles = (s.L + kFzTile - 1) / kFzTile;
  const unsigned blocks = (unsigned)((s.P + 255) / 256);
  cudaError_t e = launch_overlapped(fuzzy_prepare_kernel, dim3(blocks), dim3(256), 0, stream, s, k, skip_done);
  if (e == cudaSuccess)
    e = launch_overlapped(fuzzy_scan_kernel<false>, dim3((unsigned)(s.P * tiles)), dim3(kFzThreads), 0, stream, s, k, tiles);
  if (e == cudaSuccess) e = launch_overlapped(fuzzy_alloc_kernel, dim3(blocks), dim3(256), 0, stream, s);
  if (e == cudaSuccess)
    e = launch_overlapped(fuzzy_scan_kernel<true>, dim3((unsigned)(s.P * tiles)), dim3(kFzThreads), 0, stream, s, k, tiles);
  return e;
}

}  // namespace sdms
