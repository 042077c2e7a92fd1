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
constexpr int kScanBuf = 1536;         // matches a scanning CTA collects before it hands them over
__device__ __forceinline__ uint32_t last_bit(int32_t tok) { return ((uint32_t)tok * 2654435761u) >> 17; }
__device__ __forceinline__ uint32_t last_bit2(int32_t tok) { return ((uint32_t)tok * 0x85ebca6bu + 0x9e3779b9u) >> 17; }
static_assert(kLastBits == 1 << 15, "last_bit yields 15 bits");

// The tokens a thread fetches of tile T of prompt g (tiles are numbered path-major): four consecutive
// ones, plus one of the sixteen before the tile.  Nothing is fetched beyond the path's length.
struct TileRegs { int32_t t[4]; int32_t halo; };
__device__ __forceinline__ TileRegs fetch_tile(const Dev& s, int g, int jn, int tile, const int32_t* len_of) {
  TileRegs r;
  r.t[0] = r.t[1] = r.t[2] = r.t[3] = -1; r.halo = -1;
  if (jn >= s.N) return r;
  const int j = g * s.N + jn, t0 = tile * kScanTile;
  const int len = len_of[jn];
  const int32_t* row = s.tok + (size_t)j * s.L;
  const int x = t0 + 4 * (int)threadIdx.x;
  if (x < len) {
    if ((s.L & 3) == 0) {
      const int4 q = __ldg(reinterpret_cast<const int4*>(row + x));     // may run past len inside the row: unused there
      r.t[0] = q.x; r.t[1] = q.y; r.t[2] = q.z; r.t[3] = q.w;
    } else {
#pragma unroll
      for (int u = 0; u < 4; ++u) if (x + u < s.L) r.t[u] = __ldg(row + x + u);
    }
  }
  if (threadIdx.x < kHalo && t0 < len) {
    const int idx = t0 - kHalo + (int)threadIdx.x;
    if (idx >= 0) r.halo = __ldg(row + idx);
  }
  return r;
}

// CTA c of prompt g (blockIdx.x = g * ctas + c) walks tiles c, c + ctas, ... of that prompt (all paths of the
// prompt, tile after tile).  The set of the prompt's scan queries is built once per CTA; the next
// tile is already on its way from memory while the current one is searched.  With as many CTAs as
// tiles this is one tile per CTA (small prompts: shortest latency); with fewer it streams.
__global__ void __launch_bounds__(kScanThreads, 6) scan_kernel(Dev s, int k, int ctas, int set_slots) {
  grid_wait();
  grid_release();
  const int g = blockIdx.x / ctas, first = blockIdx.x - g * ctas;
  if (s.g_nscan[g] == 0) return;
  const int ntiles = (s.L + kScanTile - 1) / kScanTile, total = s.N * ntiles;

  __shared__ __align__(16) int32_t sh_tok[kHalo + kScanTile];
  // per-query arrays and the query set are sized by this prompt's N (dynamic shared memory), not by the
  // largest N the library takes: more CTAs fit an SM
  extern __shared__ __align__(16) int32_t scan_dyn[];
  int32_t* const sh_qid = scan_dyn;
  uint32_t* const sh_qfp = reinterpret_cast<uint32_t*>(scan_dyn + s.N);
  int32_t* const sh_cnt = scan_dyn + 2 * s.N;
  int32_t* const sh_base = scan_dyn + 3 * s.N;
  int32_t* const sh_len = scan_dyn + 4 * s.N;
  int32_t* const sh_set = scan_dyn + 5 * s.N;      // set_slots entries, a power of two >= 2 N
  __shared__ uint32_t sh_last[kLastBits / 32];   // which last tokens (hashed to 15 bits) any scan query ends in
  __shared__ int sh_nq;
  for (int n = threadIdx.x; n < s.N; n += blockDim.x) sh_len[n] = s.len[g * s.N + n];
  __syncthreads();
  // (path, tile) of the CTA's current tile and of the one after it; they advance by `ctas` tiles without a division
  const int step_j = ctas / ntiles, step_t = ctas - step_j * ntiles;
  int jn = first / ntiles, tile = first - jn * ntiles;
  int jn_next = jn + step_j, tile_next = tile + step_t;
  if (tile_next >= ntiles) { tile_next -= ntiles; ++jn_next; }
  TileRegs regs = fetch_tile(s, g, jn, tile, sh_len);                 // in flight during the set-up
  if (threadIdx.x == 0) sh_nq = 0;
  for (int x = threadIdx.x; x < set_slots; x += blockDim.x) sh_set[x] = -1;
  for (int x = threadIdx.x; x < kLastBits / 32; x += blockDim.x) sh_last[x] = 0u;
  __syncthreads();
  // the prompt's scan queries
  for (int n = threadIdx.x; n < s.N; n += blockDim.x) {
    const int i = g * s.N + n;
    if (s.q_mode[i] == Q_SCAN) {
      const int sl = atomicAdd(&sh_nq, 1);
      const uint32_t fp = s.q_fp[i];
      sh_qid[sl] = i;
      sh_qfp[sl] = fp;
      sh_cnt[sl] = 0;
      uint32_t hs = (fp >> 1) & (set_slots - 1);
      while (atomicCAS(&sh_set[hs], -1, sl) != -1) hs = (hs + 1) & (set_slots - 1);
      const int32_t* rec = s.rec + (size_t)i * kRecWords;             // rec[1 + t] = token t places from the end
      const uint32_t lb = last_bit(rec[1]), lb2 = last_bit2(rec[1]);   // two bits per query token: few false alarms
      atomicOr(&sh_last[lb >> 5], 1u << (lb & 31));
      atomicOr(&sh_last[lb2 >> 5], 1u << (lb2 & 31));
    }
  }
  __syncthreads();
  const int nq = sh_nq;
  if (nq == 0) return;

  // Matches are collected in shared memory over many tiles and handed to the match lists in one go:
  // a tile then costs two barriers and no round trip to memory.
  __shared__ uint16_t sh_bq[kScanBuf];             // query slot of a collected match
  __shared__ int32_t sh_bpos[kScanBuf];            // its position j * L + e
  __shared__ int sh_nbuf, sh_over;
  if (threadIdx.x == 0) { sh_nbuf = 0; sh_over = 0; }
  __syncthreads();

  // hands the collected matches [0, n) over: count per query, reserve a range of each list, write
  auto flush = [&](int n) {
    for (int x = threadIdx.x; x < n; x += blockDim.x) atomicAdd(&sh_cnt[sh_bq[x]], 1);
    __syncthreads();
    for (int sl = threadIdx.x; sl < nq; sl += blockDim.x) {
      const int c = sh_cnt[sl];
      sh_base[sl] = c ? atomicAdd(&s.q_cursor[sh_qid[sl]], c) : 0;
      sh_cnt[sl] = 0;
    }
    __syncthreads();
    for (int x = threadIdx.x; x < n; x += blockDim.x) {
      const int sl = sh_bq[x], i = sh_qid[sl];
      const int at = sh_base[sl] + atomicAdd(&sh_cnt[sl], 1);
      if (at < s.q_reserved[i]) s.matches[(size_t)s.q_off[i] + at] = sh_bpos[x];
      else atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
    }
    __syncthreads();
    for (int sl = threadIdx.x; sl < nq; sl += blockDim.x) sh_cnt[sl] = 0;
    if (threadIdx.x == 0) sh_nbuf = 0;
    __syncthreads();
  };

  // Calls visit(slot of the query, position e) for every match of the tile at position e = t0 + r * kScanThreads + tid.
  auto matches_at = [&](int j, int t0, int e, auto visit) {
    const int32_t* w = sh_tok + kHalo + (e - t0) - (k - 1);
    const uint32_t lb = last_bit(w[k - 1]);
    if (!(sh_last[lb >> 5] >> (lb & 31) & 1u)) return;           // no query ends in this token: nothing to hash
    const uint32_t lb2 = last_bit2(w[k - 1]);
    if (!(sh_last[lb2 >> 5] >> (lb2 & 31) & 1u)) return;
    uint64_t h = gram_init(k);
    for (int t = 0; t < k; ++t) h = gram_step(h, w[t]);
    const uint32_t fp = gram_fp(gram_final(h));
    uint32_t hs = (fp >> 1) & (set_slots - 1);
    for (int sl; (sl = sh_set[hs]) != -1; hs = (hs + 1) & (set_slots - 1)) {
      if (sh_qfp[sl] != fp) continue;
      const int i = sh_qid[sl];
      if (i == j) continue;                                       // a path never searches itself
      const int32_t* rec = s.rec + (size_t)i * kRecWords;       // the query: rec[1 + t] = token t places from the end
      bool same = true;
      for (int t = 0; t < k; ++t) same = same && (w[t] == __ldg(rec + k - t));
      if (same) visit(sl);
    }
  };
  constexpr int kPer = kScanTile / kScanThreads;

  for (int T = first; T < total; T += ctas) {
    const int j = g * s.N + jn, t0 = tile * kScanTile;
    const int e_lo = max(t0, k - 1);
    const int e_hi = min(t0 + kScanTile - 1, sh_len[jn] - 2);   // inclusive; needs one follower
    const int held = sh_nbuf;                                    // (a barrier lies between this and the last change)
    // the tile lands in shared memory; the next one is asked for before this one is looked at
    *reinterpret_cast<int4*>(sh_tok + kHalo + 4 * threadIdx.x) = make_int4(regs.t[0], regs.t[1], regs.t[2], regs.t[3]);
    if (threadIdx.x < kHalo) sh_tok[threadIdx.x] = regs.halo;
    __syncthreads();
    regs = fetch_tile(s, g, jn_next, tile_next, sh_len);
    jn = jn_next; tile = tile_next;
    jn_next += step_j; tile_next += step_t;
    if (tile_next >= ntiles) { tile_next -= ntiles; ++jn_next; }
    if (e_lo <= e_hi) {
#pragma unroll
      for (int r = 0; r < kPer; ++r) {
        const int e = t0 + r * kScanThreads + threadIdx.x;
        if (e < e_lo || e > e_hi) continue;
        matches_at(j, t0, e, [&](int sl) {
          const int at = atomicAdd(&sh_nbuf, 1);
          if (at < kScanBuf) { sh_bq[at] = (uint16_t)sl; sh_bpos[at] = j * s.L + e; }
          else sh_over = 1;
        });
      }
    }
    __syncthreads();
    if (sh_over) {
      // (same for the whole CTA) this tile's matches did not fit: hand over what was there before the
      // tile, then take the tile again with exact counts, straight into the match lists
      flush(held);
      if (threadIdx.x == 0) sh_over = 0;
#pragma unroll
      for (int r = 0; r < kPer; ++r) {
        const int e = t0 + r * kScanThreads + threadIdx.x;
        if (e >= e_lo && e <= e_hi) matches_at(j, t0, e, [&](int sl) { atomicAdd(&sh_cnt[sl], 1); });
      }
      __syncthreads();
      for (int sl = threadIdx.x; sl < nq; sl += blockDim.x) {
        const int c = sh_cnt[sl];
        sh_base[sl] = c ? atomicAdd(&s.q_cursor[sh_qid[sl]], c) : 0;
        sh_cnt[sl] = 0;
      }
      __syncthreads();
#pragma unroll
      for (int r = 0; r < kPer; ++r) {
        const int e = t0 + r * kScanThreads + threadIdx.x;
        if (e >= e_lo && e <= e_hi) matches_at(j, t0, e, [&](int sl) {
          const int i = sh_qid[sl];
          const int at = sh_base[sl] + atomicAdd(&sh_cnt[sl], 1);
          if (at < s.q_reserved[i]) s.matches[(size_t)s.q_off[i] + at] = j * s.L + e;
          else atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
        });
      }
      __syncthreads();
      for (int sl = threadIdx.x; sl < nq; sl += blockDim.x) sh_cnt[sl] = 0;
      __syncthreads();
    } else if (sh_nbuf > kScanBuf / 2) {
      flush(sh_nbuf);
    }
  }
  flush(sh_nbuf);
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
  const size_t dyn = ((size_t)5 * s.N + set_slots) * 4;
  return launch_overlapped(scan_kernel, dim3((unsigned)(ctas * s.G)), dim3(kScanThreads), dyn, stream, s, k, (int)ctas,
                           set_slots);
}

cudaError_t launch_compact_matches(const Dev& s, int32_t* offsets, int32_t* gpos, size_t cap, cudaStream_t stream) {
  compact_matches_kernel<<<1, kProbeThreads, 0, stream>>>(s, offsets, gpos, cap);
  return cudaGetLastError();
}

}  // namespace sdms
