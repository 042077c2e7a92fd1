// Cross-path suffix match (Eq. 3).
//
// probe_kernel : one thread per query path.  Hashes the path's last k tokens,
//                finds the bucket of that k-gram in the prompt's table and reads
//                its occurrence count.  The count is an upper bound on the number
//                of matches, so it sizes the query's slice of the match list.
//                Up to kInlineSlots occurrences are stored in the bucket itself:
//                such queries are answered here, from one 32-byte sector.  The
//                others are handed to the scan.
// scan_kernel  : one CTA per 1024-token tile of one path.  The tile is staged in
//                shared memory with 128-bit loads; the fingerprints of the
//                prompt's scan queries sit in a small shared hash set; every
//                position hashes its k-gram, probes the set and verifies hits
//                token by token.  Matches are counted per query in shared
//                memory, one global atomic per (CTA, query) reserves the output
//                range, and a second pass writes the positions.
#include "sdms_internal.h"
#include <algorithm>

namespace sdms {

namespace {

constexpr int kProbeThreads = 1024;

__device__ __forceinline__ long long block_exclusive_scan(long long v, long long* warp_tot, long long* total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  long long x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const long long y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) warp_tot[wid] = x;
  __syncthreads();
  if (wid == 0) {
    long long w = lane < (int)(blockDim.x >> 5) ? warp_tot[lane] : 0;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const long long y = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += y;
    }
    warp_tot[lane] = w;                       // inclusive over warps
  }
  __syncthreads();
  const long long before = wid ? warp_tot[wid - 1] : 0;
  *total = warp_tot[(blockDim.x >> 5) - 1];
  return before + x - v;
}

__global__ void __launch_bounds__(kProbeThreads) probe_kernel(Dev s, int k) {
  grid_wait();
  grid_release();
  __shared__ long long warp_tot[32];
  __shared__ long long sh_carry;
  for (int g = threadIdx.x; g < s.G; g += blockDim.x) s.g_nscan[g] = 0;
  if (threadIdx.x == 0) sh_carry = 0;
  __syncthreads();
  for (int base = 0; base < s.P; base += blockDim.x) {
    const int i = base + threadIdx.x;
    int mode = Q_NONE;
    uint32_t fp = 0, count = 0;
    const uint32_t* bucket = nullptr;
    int len_i = 0, g = 0;
    if (i < s.P) {
      len_i = s.len[i];
      g = i / s.N;
      if (len_i >= k && len_i < s.L) {
        const int32_t* q = s.tok + (size_t)i * s.L + (len_i - k);
        uint64_t h = gram_init(k);
        for (int t = 0; t < k; ++t) h = gram_step(h, q[t]);
        h = gram_final(h);
        fp = gram_fp(h);
        const uint32_t* table = index_table(s, g, k);
        uint32_t b = gram_bucket(h, s.table_cap);
        for (uint32_t probe = 0; probe < s.table_cap; ++probe) {
          const uint32_t* cand = table + (size_t)b * kBucketWords;
          const uint32_t w0 = cand[0];
          if (w0 == fp) { bucket = cand; break; }
          if (w0 == 0u) break;
          b = (b + 1) & (s.table_cap - 1);
        }
        if (bucket) {
          count = bucket[1];
          mode = count <= (uint32_t)kInlineSlots ? Q_INLINE : Q_SCAN;
        }
      }
    }
    long long total;
    const long long off = sh_carry + block_exclusive_scan((long long)count, warp_tot, &total);
    if (mode != Q_NONE && off + (long long)count > s.match_cap) {
      mode = Q_NONE;
      atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
    }
    if (i < s.P) {
      int written = 0;
      if (mode == Q_INLINE) {
        const int32_t* q = s.tok + (size_t)i * s.L + (len_i - k);
        for (uint32_t sl = 0; sl < count; ++sl) {
          const uint32_t lpos = bucket[2 + sl];
          const int j = g * s.N + (int)(lpos / (uint32_t)s.L);
          const int e = (int)(lpos % (uint32_t)s.L);
          if (j == i || e > s.len[j] - 2) continue;
          const int32_t* c = s.tok + (size_t)j * s.L + (e - k + 1);
          bool same = true;
          for (int t = 0; t < k; ++t) same = same && (c[t] == q[t]);
          if (same) s.matches[off + written++] = j * s.L + e;
        }
      } else if (mode == Q_SCAN) {
        atomicAdd(&s.g_nscan[g], 1);
      }
      s.q_fp[i] = fp;
      s.q_mode[i] = mode;
      s.q_reserved[i] = mode == Q_NONE ? 0 : (int32_t)count;
      s.q_off[i] = (int32_t)(off < s.match_cap ? off : s.match_cap);
      s.q_cursor[i] = written;
    }
    __syncthreads();
    if (threadIdx.x == 0) sh_carry += total;
    __syncthreads();
  }
}

constexpr int kLastBits = 32768;       // a prompt has up to 1024 scan queries: the reject test must stay selective
constexpr unsigned FULL_MASK = 0xffffffffu;
constexpr int kWarpBuf = 96;           // matches a warp of a scanning CTA collects before it hands them over
__device__ __forceinline__ uint32_t last_bit(int32_t tok) { return ((uint32_t)tok * 2654435761u) >> 17; }
__device__ __forceinline__ uint32_t last_bit2(int32_t tok) { return ((uint32_t)tok * 0x85ebca6bu + 0x9e3779b9u) >> 17; }
static_assert(kLastBits == 1 << 15, "last_bit yields 15 bits");
static_assert(kScanTile == 4 * kScanThreads, "a thread looks at the four tokens it fetched");

// The four consecutive tokens a thread fetches of tile `tile` of path jn of prompt g.  Nothing is
// fetched beyond the path's length (-1 stands for "no token").
struct TileRegs { int32_t t[4]; };
__device__ __forceinline__ TileRegs fetch_tile(const Dev& s, int g, int jn, int tile, const int32_t* len_of) {
  TileRegs r;
  r.t[0] = r.t[1] = r.t[2] = r.t[3] = -1;
  if (jn >= s.N) return r;
  const int32_t* row = s.tok + (size_t)(g * s.N + jn) * s.L;
  const int x = tile * kScanTile + 4 * (int)threadIdx.x;
  if (x < len_of[jn]) {
    if ((s.L & 3) == 0) {
      const int4 q = __ldg(reinterpret_cast<const int4*>(row + x));     // may run past the length inside the row: unused there
      r.t[0] = q.x; r.t[1] = q.y; r.t[2] = q.z; r.t[3] = q.w;
    } else {
#pragma unroll
      for (int u = 0; u < 4; ++u) if (x + u < s.L) r.t[u] = __ldg(row + x + u);
    }
  }
  return r;
}

// CTA c of prompt g (blockIdx.x = g * ctas + c) walks tiles c, c + ctas, ... of that prompt (all paths of the
// prompt, tile after tile).  The set of the prompt's scan queries is built once per CTA.  After that
// the warps run on their own, without CTA barriers: a thread filters the four tokens it fetched in
// registers (two hashed bits of the set of the queries' last tokens) while the next tile is already on
// its way; only a token that passes reads its window, from memory that is in cache by then.  Matches
// go to a small buffer per warp that the warp hands over itself.  With as many CTAs as tiles this is
// one tile per CTA (small prompts: shortest latency); with fewer it streams.
__global__ void __launch_bounds__(kScanThreads, 6) scan_kernel(Dev s, int k, int ctas, int set_slots) {
  grid_wait();
  grid_release();
  const int g = blockIdx.x / ctas, first = blockIdx.x - g * ctas;
  if (s.g_nscan[g] == 0) return;
  const int ntiles = (s.L + kScanTile - 1) / kScanTile, total = s.N * ntiles;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // per-query arrays and the query set are sized by this prompt's N (dynamic shared memory)
  extern __shared__ __align__(16) int32_t scan_dyn[];
  int32_t* const sh_qid = scan_dyn;
  uint32_t* const sh_qfp = reinterpret_cast<uint32_t*>(scan_dyn + s.N);
  int32_t* const sh_len = scan_dyn + 2 * s.N;
  int32_t* const sh_set = scan_dyn + 3 * s.N;      // set_slots entries, a power of two >= 2 N
  __shared__ uint32_t sh_last[kLastBits / 32];     // which last tokens (hashed to 15 bits, twice) any scan query ends in
  __shared__ uint16_t sh_wq[kScanThreads / 32][kWarpBuf];   // per warp: query slot of a collected match
  __shared__ int32_t sh_wpos[kScanThreads / 32][kWarpBuf];  // ... and its position j * L + e
  __shared__ int sh_wn[kScanThreads / 32];
  __shared__ int sh_nq;
  for (int n = threadIdx.x; n < s.N; n += blockDim.x) sh_len[n] = s.len[g * s.N + n];
  if (threadIdx.x == 0) sh_nq = 0;
  if (threadIdx.x < kScanThreads / 32) sh_wn[threadIdx.x] = 0;
  for (int x = threadIdx.x; x < set_slots; x += blockDim.x) sh_set[x] = -1;
  for (int x = threadIdx.x; x < kLastBits / 32; x += blockDim.x) sh_last[x] = 0u;
  __syncthreads();
  // (path, tile) of the CTA's current tile and of the one after it; they advance by `ctas` tiles without a division
  const int step_j = ctas / ntiles, step_t = ctas - step_j * ntiles;
  int jn = first / ntiles, tile = first - jn * ntiles;
  int jn_next = jn + step_j, tile_next = tile + step_t;
  if (tile_next >= ntiles) { tile_next -= ntiles; ++jn_next; }
  TileRegs regs = fetch_tile(s, g, jn, tile, sh_len);                 // in flight during the set-up
  // the prompt's scan queries
  for (int n = threadIdx.x; n < s.N; n += blockDim.x) {
    const int i = g * s.N + n;
    if (s.q_mode[i] == Q_SCAN) {
      const int sl = atomicAdd(&sh_nq, 1);
      const uint32_t fp = s.q_fp[i];
      sh_qid[sl] = i;
      sh_qfp[sl] = fp;
      uint32_t hs = (fp >> 1) & (set_slots - 1);
      while (atomicCAS(&sh_set[hs], -1, sl) != -1) hs = (hs + 1) & (set_slots - 1);
      const int32_t last = s.rec[(size_t)i * kRecWords + 1];
      const uint32_t lb = last_bit(last), lb2 = last_bit2(last);      // two bits per query token: few false alarms
      atomicOr(&sh_last[lb >> 5], 1u << (lb & 31));
      atomicOr(&sh_last[lb2 >> 5], 1u << (lb2 & 31));
    }
  }
  __syncthreads();
  if (sh_nq == 0) return;
  // from here on no CTA barrier: every warp goes through the same tiles at its own pace

  // one entry of the match list of query slot sl (the list's cursor is bumped by one)
  auto emit = [&](int sl, int pos) {
    const int i = sh_qid[sl];
    const int at = atomicAdd(&s.q_cursor[i], 1);
    if (at < s.q_reserved[i]) s.matches[(size_t)s.q_off[i] + at] = pos;
    else atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
  };
  // the warp hands its collected matches over; lanes with the same query share one bump of its cursor
  auto flush_warp = [&]() {
    __syncwarp();
    const int n = min(sh_wn[warp], kWarpBuf);
    for (int x0 = 0; x0 < n; x0 += 32) {
      const int x = x0 + lane;
      const bool on = x < n;
      const int sl = on ? sh_wq[warp][x] : -1 - lane;
      const unsigned same = __match_any_sync(FULL_MASK, sl);
      const int leader = __ffs(same) - 1;
      int base = 0;
      if (on && lane == leader) base = atomicAdd(&s.q_cursor[sh_qid[sl]], __popc(same));
      base = __shfl_sync(FULL_MASK, base, leader);
      if (on) {
        const int i = sh_qid[sl];
        const int at = base + __popc(same & ((1u << lane) - 1u));
        if (at < s.q_reserved[i]) s.matches[(size_t)s.q_off[i] + at] = sh_wpos[warp][x];
        else atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
      }
    }
    __syncwarp();
    if (lane == 0) sh_wn[warp] = 0;
    __syncwarp();
  };

  for (int T = first; T < total; T += ctas) {
    const int j = g * s.N + jn, t0 = tile * kScanTile;
    const int e_lo = max(t0, k - 1);
    const int e_hi = min(t0 + kScanTile - 1, sh_len[jn] - 2);   // inclusive; needs one follower
    const int32_t* row = s.tok + (size_t)j * s.L;
    const TileRegs cur = regs;
    regs = fetch_tile(s, g, jn_next, tile_next, sh_len);         // the next tile is asked for before this one is looked at
    jn = jn_next; tile = tile_next;
    jn_next += step_j; tile_next += step_t;
    if (tile_next >= ntiles) { tile_next -= ntiles; ++jn_next; }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = t0 + 4 * (int)threadIdx.x + u;
      if (e < e_lo || e > e_hi) continue;
      const int32_t tok = cur.t[u];
      const uint32_t lb = last_bit(tok);
      if (!(sh_last[lb >> 5] >> (lb & 31) & 1u)) continue;       // no query ends in this token: nothing to hash
      const uint32_t lb2 = last_bit2(tok);
      if (!(sh_last[lb2 >> 5] >> (lb2 & 31) & 1u)) continue;
      // the window that ends at e (its tokens are in cache: this thread or its neighbours just fetched them)
      const int32_t* w = row + e - (k - 1);
      uint64_t h = gram_init(k);
      for (int t = 0; t < k - 1; ++t) h = gram_step(h, __ldg(w + t));
      h = gram_step(h, tok);
      const uint32_t fp = gram_fp(gram_final(h));
      uint32_t hs = (fp >> 1) & (set_slots - 1);
      for (int sl; (sl = sh_set[hs]) != -1; hs = (hs + 1) & (set_slots - 1)) {
        if (sh_qfp[sl] != fp) continue;
        const int i = sh_qid[sl];
        if (i == j) continue;                                     // a path never searches itself
        const int32_t* rec = s.rec + (size_t)i * kRecWords;       // the query: rec[1 + t] = token t places from the end
        bool same = true;
        for (int t = 0; t < k; ++t) same = same && (__ldg(w + t) == __ldg(rec + k - t));
        if (!same) continue;
        const int at = atomicAdd(&sh_wn[warp], 1);
        if (at < kWarpBuf) { sh_wq[warp][at] = (uint16_t)sl; sh_wpos[warp][at] = j * s.L + e; }
        else emit(sl, j * s.L + e);                               // the buffer is full: straight to the list
      }
    }
    __syncwarp();
    if (sh_wn[warp] > kWarpBuf / 2) flush_warp();                 // same for the whole warp
  }
  flush_warp();
}

// Inspection only: packs the per-query slices of the match list.
__global__ void __launch_bounds__(kProbeThreads) compact_matches_kernel(Dev s, int32_t* offsets, int32_t* gpos,
                                                                        size_t cap) {
  __shared__ long long warp_tot[32];
  __shared__ long long sh_carry;
  if (threadIdx.x == 0) sh_carry = 0;
  __syncthreads();
  for (int base = 0; base < s.P; base += blockDim.x) {
    const int i = base + threadIdx.x;
    long long m = 0;
    if (i < s.P && s.q_mode[i] != Q_NONE) m = min(s.q_cursor[i], s.q_reserved[i]);
    long long total;
    const long long off = sh_carry + block_exclusive_scan(m, warp_tot, &total);
    if (i < s.P) offsets[i] = (int32_t)off;
    __syncthreads();
    if (threadIdx.x == 0) sh_carry += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) offsets[s.P] = (int32_t)sh_carry;
  __syncthreads();
  for (int i = 0; i < s.P; ++i) {
    const int m = offsets[i + 1] - offsets[i];
    for (int x = threadIdx.x; x < m; x += blockDim.x)
      if ((size_t)(offsets[i] + x) < cap) gpos[offsets[i] + x] = s.matches[(size_t)s.q_off[i] + x];
  }
}

}  // namespace

cudaError_t launch_probe(const Dev& s, int k, cudaStream_t stream) {
  return launch_overlapped(probe_kernel, dim3(1), dim3(kProbeThreads), 0, stream, s, k);
}

cudaError_t launch_scan(const Dev& s, int k, cudaStream_t stream) {
  // one CTA per tile while that keeps the device busy for one round; beyond that each CTA streams
  // through its share of its prompt's tiles
  const long long per_prompt = (long long)s.N * ((s.L + kScanTile - 1) / kScanTile);
  const long long budget = 148LL * 8 * 4;
  long long ctas = per_prompt;
  if ((long long)s.G * per_prompt > budget) ctas = std::max(1LL, std::min(per_prompt, budget / s.G));
  int set_slots = 64;
  while (set_slots < 2 * s.N) set_slots *= 2;
  const size_t dyn = ((size_t)3 * s.N + set_slots) * 4;
  return launch_overlapped(scan_kernel, dim3((unsigned)(ctas * s.G)), dim3(kScanThreads), dyn, stream, s, k, (int)ctas,
                           set_slots);
}

cudaError_t launch_compact_matches(const Dev& s, int32_t* offsets, int32_t* gpos, size_t cap, cudaStream_t stream) {
  compact_matches_kernel<<<1, kProbeThreads, 0, stream>>>(s, offsets, gpos, cap);
  return cudaGetLastError();
}

}  // namespace sdms
