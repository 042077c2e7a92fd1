// Cross-path suffix match (Eq. 3).
//
// probe_kernel : one thread per query path.  Hashes the path's last k tokens,
//                finds the bucket of that k-gram in the prompt's table and reads
//                its occurrence count.  The count is an upper bound on the number
//                of matches, so it sizes the query's slice of the match list.
//                Up to kInlineSlots occurrences are stored in the bucket itself:
//                such queries are answered here, from one 32-byte sector.  The
//                others are handed to the scan.
// scan_kernel  : the histories of a prompt are read once, in tiles, for all of
//                its scan queries together.  A token is first tested against a
//                bit table of the queries' last tokens; the few positions that
//                pass are queued per warp and looked at 32 at a time (window
//                hash, probe of the prompt's query set, verification token by
//                token).  Small prompts: one CTA per 1024-token tile, tokens
//                fetched with 128-bit loads.  Stores of many tiles: each CTA
//                streams 2048-token tiles through shared-memory stages filled
//                by bulk copies.
#include "sdms_internal.h"
#include <algorithm>

namespace sdms {

namespace {

constexpr int kProbeThreads = 1024;
constexpr unsigned FULL_MASK = 0xffffffffu;

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

// One warp per query path.  The path's record (length and newest tokens, one 128-byte line) gives the
// query; the warp looks at four neighbouring buckets of the k-gram's table at a time (eight lanes per
// bucket, one round trip).  A k-gram with at most kInlineSlots occurrences is answered here: lane sl
// checks occurrence sl (other path, a follower exists, tokens equal) and the matches go to the
// query's own kInlineArea slots at the front of the match list.  Any other query reserves as many slots
// as the k-gram has occurrences behind that area (one atomic on a cursor that the build's last kernel
// leaves at zero) and is handed to the scan.  Slices therefore lie in no particular order.
constexpr int kProbeWarps = 8;
constexpr int kInlineArea = 8;
static_assert(kInlineArea >= kInlineSlots && kRecWords == 32 && kBucketWords == 8, "lane layout of the probe");

__global__ void __launch_bounds__(kProbeWarps * 32) probe_kernel(Dev s, int k, int skip_done) {
  grid_wait();
  grid_release();
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * kProbeWarps + (threadIdx.x >> 5);
  if (i >= s.P) return;                                          // whole warps
  if (skip_done && s.q_mode[i] == Q_DONE) return;                // back-off: this path has its matches from a longer suffix
  const int g = i / s.N;
  const int32_t mine = s.rec[(size_t)i * kRecWords + lane];
  const int len_i = __shfl_sync(FULL_MASK, mine, 0);
  int mode = Q_NONE, written = 0, off = i * kInlineArea;
  uint32_t fp = 0, count = 0;
  if (len_i >= k && len_i < s.L) {
    // the query, oldest token first: token x of it sits in lane k - x of the record
    // fp names the whole k-gram (the scan looks queries up by it); the index is asked for the last nx tokens
    const int nx = min(k, s.idx_n);
    uint64_t h = gram_init(k), hx = gram_init(nx);
    for (int x = 0; x < k; ++x) {
      const int32_t t = __shfl_sync(FULL_MASK, mine, k - x);
      h = gram_step(h, t);
      if (x >= k - nx) hx = gram_step(hx, t);
    }
    fp = gram_fp(gram_final(h));
    hx = gram_final(hx);
    const uint32_t want = gram_fp(hx);
    const uint32_t* table = index_table(s, g, nx);
    uint32_t b = gram_bucket(hx, s.table_cap);
    int found = -1;                                              // lane that holds the bucket's first word
    uint32_t word = 0;
    for (uint32_t probe = 0; probe < s.table_cap && found < 0; probe += 4) {
      const uint32_t bb = (b + (lane >> 3)) & (s.table_cap - 1);
      word = table[(size_t)bb * kBucketWords + (lane & 7)];
      bool end = false;
      for (int r = 0; r < 4 && found < 0 && !end; ++r) {
        const uint32_t w0 = __shfl_sync(FULL_MASK, word, 8 * r);
        if (w0 == want) found = 8 * r;
        else if (w0 == 0u) end = true;
      }
      if (end) break;
      b = (b + 4) & (s.table_cap - 1);
    }
    if (found >= 0) {
      count = __shfl_sync(FULL_MASK, word, found + 1);
      mode = count <= (uint32_t)kInlineSlots ? Q_INLINE : Q_SCAN;
      if (mode == Q_INLINE) {
        const uint32_t lpos = __shfl_sync(FULL_MASK, word, found + 2 + (lane < kInlineSlots ? lane : 0));
        bool same = false;
        int gpos = 0;
        if (lane < (int)count) {
          const int jn = (int)(lpos / (uint32_t)s.L);
          const int j = g * s.N + jn, e = (int)(lpos - (uint32_t)jn * (uint32_t)s.L);
          gpos = j * s.L + e;
          if (j != i && e >= k - 1) {
            const int len_j = s.len[j];
            const int32_t* c = s.tok + (size_t)j * s.L + (e - k + 1);
            const int32_t* q = s.tok + (size_t)i * s.L + (len_i - k);
            same = true;
            for (int t = 0; t < k; ++t) same = same && (c[t] == q[t]);          // no early exit: the loads go out together
            same = same && e <= len_j - 2;
          }
        }
        const unsigned ok = __ballot_sync(FULL_MASK, same);
        written = __popc(ok);
        if ((long long)off + kInlineArea > s.match_cap) {
          if (lane == 0) atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
          mode = Q_NONE; written = 0;
        } else if (same) {
          s.matches[off + __popc(ok & ((1u << lane) - 1u))] = gpos;
        }
      } else {
        long long at = 0;
        if (lane == 0) at = (long long)atomicAdd(s.match_cursor, (unsigned long long)count) + (long long)s.P * kInlineArea;
        at = __shfl_sync(FULL_MASK, at, 0);
        if (at + (long long)count > s.match_cap) {
          if (lane == 0) atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
          mode = Q_NONE;
        } else {
          off = (int)at;
          if (lane == 0) atomicAdd(&s.g_nscan[g], 1);
        }
      }
    }
  }
  if (lane == 0) {
    s.q_fp[i] = fp;
    s.q_mode[i] = mode;
    s.q_reserved[i] = mode == Q_NONE ? 0 : (mode == Q_INLINE ? kInlineArea : (int32_t)count);
    s.q_off[i] = off;
    s.q_cursor[i] = written;
  }
}

// Reject test on a position's own token: one bit in each of two tables, set for the last token of every
// scan query of the prompt (up to 1024 of them).  The first table is looked at for every token, the
// second only for the few that pass the first.
constexpr int kLastBits = 65536;
constexpr int kLast2Bits = 8192;
constexpr int kCandBuf = 64;           // entries a warp may have waiting: fewer than 32 left over plus one per lane
__device__ __forceinline__ uint32_t last_bit(int32_t tok) { return ((uint32_t)tok * 2654435761u) >> 16; }
__device__ __forceinline__ uint32_t last_bit2(int32_t tok) { return ((uint32_t)tok * 0x85ebca6bu + 0x9e3779b9u) >> 19; }
static_assert(kLastBits == 1 << 16 && kLast2Bits == 1 << 13, "last_bit yields 16 bits, last_bit2 13");
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

// ---- bulk-copy staging for the streaming form of the scan -------------------------------------
// A CTA that walks many tiles keeps kStreamStages of them in flight as bulk copies (the copy engine
// writes a whole 4 KB tile into shared memory and signals an mbarrier), so the bytes in flight do not
// depend on registers or on how many warps are resident.
constexpr int kStreamStages = 4;
constexpr int kStreamTile = 2 * kScanTile;           // tokens per stage: a thread takes eight of them
constexpr int kStreamThreads = kScanThreads + 32;   // eight scanning warps and one warp that issues the copies
constexpr int kStreamSmemMax = 96 * 1024;             // dynamic shared memory the streaming form may ask for
constexpr long long kWaitCycles = 400000000LL;       // about a fifth of a second (the kernel takes 20-140 us): a wait that long has failed

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Waits for the phase with the given parity to complete; gives up after kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try(bar, parity))
    if (clock64() - t0 > kWaitCycles) return false;
  return true;
}
// bytes (a multiple of 16, both addresses 16-byte aligned) from global to this CTA's shared memory
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

// CTA c of prompt g (blockIdx.x = g * ctas + c) walks tiles c, c + ctas, ... of that prompt (all paths of the
// prompt, tile after tile).  The set of the prompt's scan queries is built once per CTA.  After that
// the warps run on their own, without CTA barriers.  A thread tests the four tokens it holds of the
// tile against the first reject table, without a branch in between.  Positions that pass are not looked
// at there and then, by one or two lanes with the rest of the warp idle: the warp queues them in shared
// memory, and once 32 are waiting every lane takes one (second reject table, hash of the window, probe
// of the query set, token-by-token verification).  Lanes whose positions match the same query share one
// bump of that query's cursor in the match list.
// STREAM = false: a thread fetches its four tokens itself, one tile ahead.  With as many CTAs as tiles
// this is one tile per CTA (small prompts: shortest latency).
// STREAM = true : a ninth warp keeps kStreamStages tiles in flight as bulk copies into shared memory
// (full / empty mbarrier per stage); a scanning thread takes its tokens out of the stage and gives its
// share of the stage back at once.  Needs rows that start and end on 16-byte boundaries (L a multiple of 4).
template <bool STREAM>
__global__ void __launch_bounds__(STREAM ? kStreamThreads : kScanThreads, STREAM ? 4 : 6)
scan_kernel(Dev s, int k, int ctas, int set_slots) {
  const int g = blockIdx.x / ctas, first = blockIdx.x - g * ctas;
  constexpr int TILE = STREAM ? kStreamTile : kScanTile;
  const int ntiles = (s.L + TILE - 1) / TILE, total = s.N * ntiles;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool scanner = !STREAM || warp < kScanThreads / 32;

  // per-query arrays and the query set are sized by this prompt's N (dynamic shared memory)
  extern __shared__ __align__(128) int32_t scan_dyn[];
  int32_t* const sh_stage = scan_dyn;                                 // STREAM: kStreamStages tiles
  int32_t* const sh_qid = scan_dyn + (STREAM ? kStreamStages * kStreamTile : 0);
  uint32_t* const sh_qfp = reinterpret_cast<uint32_t*>(sh_qid + s.N);
  int32_t* const sh_len = sh_qid + 2 * s.N;
  int32_t* const sh_qlast = sh_qid + 3 * s.N;     // last token of the query in a slot
  int32_t* const sh_set = sh_qid + 4 * s.N;       // set_slots entries, a power of two >= 4 N
  __shared__ __align__(16) uint32_t sh_last[kLastBits / 32];     // which last tokens (hashed to 16 bits) any scan query ends in
  __shared__ __align__(16) uint32_t sh_last2[kLast2Bits / 32];   // the same under a second hash (13 bits)
  __shared__ int2 sh_cand[kScanThreads / 32][kCandBuf];     // per warp: waiting (jn * L + e of a thread's first token, which of its four or eight)
  __shared__ int sh_nq;
  __shared__ __align__(8) uint64_t sh_full[kStreamStages], sh_empty[kStreamStages];
  for (int n = threadIdx.x; n < s.N; n += blockDim.x) sh_len[n] = s.len[g * s.N + n];
  if (threadIdx.x == 0) sh_nq = 0;
  for (int x = threadIdx.x; x < set_slots; x += blockDim.x) sh_set[x] = -1;
  for (int x = threadIdx.x; x < kLastBits / 128; x += blockDim.x) reinterpret_cast<uint4*>(sh_last)[x] = make_uint4(0u, 0u, 0u, 0u);
  for (int x = threadIdx.x; x < kLast2Bits / 128; x += blockDim.x) reinterpret_cast<uint4*>(sh_last2)[x] = make_uint4(0u, 0u, 0u, 0u);
  if (STREAM && threadIdx.x == kScanThreads) {
    for (int st = 0; st < kStreamStages; ++st) { mbar_init(&sh_full[st], 1); mbar_init(&sh_empty[st], kScanThreads); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the last token of the first path this thread will look at below (path records are older than the probe too)
  const int i_pre = g * s.N + (int)threadIdx.x;
  int32_t last_pre = 0;
  if ((int)threadIdx.x < s.N) last_pre = s.rec[(size_t)i_pre * kRecWords + 1];
  // Up to here nothing was read that the probe writes (path lengths, records and tokens are older than the probe: its
  // CTAs let this kernel start only after their own wait), so the set-up above overlaps the probe's tail.
  grid_wait();
  grid_release();
  if (blockIdx.x == 0 && threadIdx.x < kWideCtlWords && s.w_grid) s.w_ctl[threadIdx.x] = 0ull;   // the wide pass of this build starts with an empty list
  // what the probe left for that path, asked for together with the prompt's count of scan queries: one round trip
  int32_t mode_pre = Q_NONE;
  uint32_t fp_pre = 0u;
  if ((int)threadIdx.x < s.N) { mode_pre = s.q_mode[i_pre]; fp_pre = s.q_fp[i_pre]; }
  if (s.g_nscan[g] == 0) return;
  __syncthreads();
  // (path, tile) of the CTA's current tile and of the one after it; they advance by `ctas` tiles without a division
  const int step_j = ctas / ntiles, step_t = ctas - step_j * ntiles;
  int jn = first / ntiles, tile = first - jn * ntiles;
  int jn_next = jn + step_j, tile_next = tile + step_t;
  if (tile_next >= ntiles) { tile_next -= ntiles; ++jn_next; }

  // STREAM: the issuing thread's own walk over the CTA's tiles.  A tile of a path that is shorter than
  // the tile's start is not copied; its barrier still completes, so that the phases stay in step.
  int pj = jn, ptile = tile, pT = first, pstage = 0;
  auto issue_tile = [&]() {
    const int t0 = ptile * TILE;
    const int have = sh_len[pj] - t0;                                 // tokens of this path from t0 on
    if (have > 0) {
      const uint32_t bytes = 4u * (uint32_t)min(TILE, min(s.L - t0, (have + 3) & ~3));
      mbar_arrive_expect(&sh_full[pstage], bytes);
      bulk_load(sh_stage + pstage * TILE, s.tok + (size_t)(g * s.N + pj) * s.L + t0, bytes, &sh_full[pstage]);
    } else {
      mbar_arrive(&sh_full[pstage]);
    }
    pT += ctas; pj += step_j; ptile += step_t;
    if (ptile >= ntiles) { ptile -= ntiles; ++pj; }
    if (++pstage == kStreamStages) pstage = 0;
  };
  int issued = 0;
  TileRegs regs;
  if (STREAM) {
    if (threadIdx.x == kScanThreads)
      for (; issued < kStreamStages && pT < total; ++issued) issue_tile();   // in flight during the set-up
  } else {
    regs = fetch_tile(s, g, jn, tile, sh_len);                        // in flight during the set-up
  }
  // the prompt's scan queries
  for (int n = threadIdx.x; n < s.N; n += blockDim.x) {
    const int i = g * s.N + n;
    const bool have = n == (int)threadIdx.x;                         // the thread's first path: already here
    if ((have ? mode_pre : s.q_mode[i]) == Q_SCAN) {
      const int sl = atomicAdd(&sh_nq, 1);
      const uint32_t fp = have ? fp_pre : s.q_fp[i];
      sh_qid[sl] = i;
      sh_qfp[sl] = fp;
      uint32_t hs = (fp >> 1) & (set_slots - 1);
      while (atomicCAS(&sh_set[hs], -1, sl) != -1) hs = (hs + 1) & (set_slots - 1);
      const int32_t last = have ? last_pre : s.rec[(size_t)i * kRecWords + 1];
      sh_qlast[sl] = last;
      const uint32_t lb = last_bit(last), lb2 = last_bit2(last);      // two bits per query token: few false alarms
      atomicOr(&sh_last[lb >> 5], 1u << (lb & 31));
      atomicOr(&sh_last2[lb2 >> 5], 1u << (lb2 & 31));
    }
  }
  __syncthreads();
  if (!STREAM && sh_nq == 0) return;
  // from here on no CTA barrier: every warp goes through the same tiles at its own pace

  if (STREAM && !scanner) {
    // the issuing warp: one thread refills a stage as soon as all scanning warps have given it back
    if (lane != 0) return;
    uint32_t round = 0;                                               // how often the stages have been refilled
    for (int st = 0; pT < total; ++issued) {
      if (!mbar_wait(&sh_empty[st], round & 1u)) { atomicOr(s.status, SDMS_STATUS_TIMEOUT); return; }
      issue_tile();
      if (++st == kStreamStages) { st = 0; ++round; }
    }
    return;
  }

  // The warp looks at waiting entries, 32 at a time (newest first), until fewer than 32 are left; with
  // `all` set, until none is left.  cn is the same in every lane.  An entry names up to four positions;
  // whether a position can end a match at all (k - 1 <= e <= len - 2) is decided here, not in the filter.
  int cn = 0;
  const uint32_t lanes_below = (1u << lane) - 1u;
  auto drain = [&](bool all) {
    __syncwarp();
    while (cn >= 32 || (all && cn > 0)) {
      const int take = min(32, cn);
      cn -= take;
      int2 ent = make_int2(0, 0);
      if (lane < take) ent = sh_cand[warp][cn + lane];
      const int jl = ent.x / s.L, e_first = ent.x - jl * s.L, j = g * s.N + jl;
      const int e_last = sh_len[jl] - 2;
      const int32_t* const row = s.tok + (size_t)j * s.L;
      uint32_t todo = (uint32_t)ent.y;
      while (__any_sync(FULL_MASK, todo != 0u)) {                  // one position of every lane's entry per round
        const int u = __ffs(todo) - 1;                              // -1: this lane has none left
        todo &= todo - 1u;
        const int e = e_first + (u & 3) + (u >> 2) * kScanTile;   // bits 4..7: the thread's second four tokens
        const bool on = u >= 0 && e >= k - 1 && e <= e_last;
        const int32_t* w = row + e - (k - 1);                       // the window that ends at e
        const int32_t tok = on ? __ldg(w + k - 1) : 0;
        const uint32_t lb2 = last_bit2(tok);
        bool live = on && (sh_last2[lb2 >> 5] >> (lb2 & 31) & 1u);
        uint32_t fp = 0u, hs = 0u;
        if (live) {
          uint64_t h = gram_init(k);
          for (int t = 0; t < k - 1; ++t) h = gram_step(h, __ldg(w + t));
          h = gram_step(h, tok);
          fp = gram_fp(gram_final(h));
          hs = (fp >> 1) & (set_slots - 1);
        }
        while (__any_sync(FULL_MASK, live)) {                      // every lane walks its probe run
          const int sl = live ? sh_set[hs] : -1;
          live = live && sl != -1;
          hs = (hs + 1) & (set_slots - 1);
          int i = -1;
          if (live && sh_qfp[sl] == fp) {
            i = sh_qid[sl];
            if (i == j) i = -1;                                    // a path never searches itself
            if (i >= 0) {
              const int32_t* rec = s.rec + (size_t)i * kRecWords; // the query: rec[1 + t] = token t places from the end
              bool same = tok == sh_qlast[sl];
              for (int t = 0; t < k - 1; ++t) same = same && (__ldg(w + t) == __ldg(rec + k - t));
              if (!same) i = -1;
            }
          }
          if (!__any_sync(FULL_MASK, i >= 0)) continue;
          const unsigned same = __match_any_sync(FULL_MASK, i >= 0 ? i : -1 - lane);
          const int leader = __ffs(same) - 1;
          int base = 0;
          if (i >= 0 && lane == leader) base = atomicAdd(&s.q_cursor[i], __popc(same));
          base = __shfl_sync(FULL_MASK, base, leader);
          if (i >= 0) {
            const int at = base + __popc(same & lanes_below);
            if (at < s.q_reserved[i]) s.matches[(size_t)s.q_off[i] + at] = j * s.L + e;
            else atomicOr(s.status, SDMS_STATUS_MATCH_OVERFLOW);
          }
        }
      }
      __syncwarp();
    }
  };

  const int tid4 = 4 * (int)threadIdx.x;
  int stage = 0;
  uint32_t phase = 0;
  for (int T = first; T < total; T += ctas) {
    const int t0 = tile * TILE, jn_now = jn;
    TileRegs cur, cur2;
    if (STREAM) {
      if (!__all_sync(FULL_MASK, mbar_wait(&sh_full[stage], phase))) {  // cannot happen; the warp leaves in an orderly way
        atomicOr(s.status, SDMS_STATUS_TIMEOUT);
        for (int it = 0; it < 10000; ++it) __nanosleep(1000);         // copies still in flight land in live shared memory
        break;
      }
      const int4* const st4 = reinterpret_cast<const int4*>(sh_stage + stage * TILE);
      const int4 q = st4[threadIdx.x], q2 = st4[kScanThreads + threadIdx.x];   // tokens e0..e0+3 and e0+1024..e0+1027
      cur.t[0] = q.x; cur.t[1] = q.y; cur.t[2] = q.z; cur.t[3] = q.w;  // beyond the copied bytes: stale, turned down in drain()
      cur2.t[0] = q2.x; cur2.t[1] = q2.y; cur2.t[2] = q2.z; cur2.t[3] = q2.w;
      mbar_arrive(&sh_empty[stage]);                                   // this thread has its tokens; when all have, the stage is refilled
      if (++stage == kStreamStages) { stage = 0; phase ^= 1u; }
    } else {
      cur = regs;
      regs = fetch_tile(s, g, jn_next, tile_next, sh_len);       // the next tile is asked for before this one is looked at
    }
    jn = jn_next; tile = tile_next;
    jn_next += step_j; tile_next += step_t;
    if (tile_next >= ntiles) { tile_next -= ntiles; ++jn_next; }
    if (t0 > sh_len[jn_now] - 2) continue;                        // nothing of the path in this tile (same for the whole CTA)
    // first reject table: bit 0 of w[u] says whether token u passes.  Almost always none does, so the
    // words are only OR-ed together; the exact mask is worked out for the few threads with a set bit.
    uint32_t wd[STREAM ? 8 : 4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t lb = last_bit(cur.t[u]);
      wd[u] = sh_last[lb >> 5] >> (lb & 31);
    }
    uint32_t any = (wd[0] | wd[1]) | (wd[2] | wd[3]);
    if (STREAM) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t lb = last_bit(cur2.t[u]);
        wd[4 + u] = sh_last[lb >> 5] >> (lb & 31);
      }
      any |= (wd[4] | wd[5]) | (wd[6] | wd[7]);
    }
    uint32_t hit = 0u;
    if (any & 1u) {
#pragma unroll
      for (int u = 0; u < (STREAM ? 8 : 4); ++u) hit |= (wd[u] & 1u) << u;
    }
    const unsigned b = __ballot_sync(FULL_MASK, hit != 0u);
    if (b) {                                                      // queue what passed
      if (hit) sh_cand[warp][cn + __popc(b & lanes_below)] = make_int2(jn_now * s.L + t0 + tid4, (int)hit);
      cn += __popc(b);
      if (cn >= 32) drain(false);
    }
  }
  drain(true);
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

cudaError_t launch_probe(const Dev& s, int k, int skip_done, cudaStream_t stream) {
  return launch_overlapped(probe_kernel, dim3((s.P + kProbeWarps - 1) / kProbeWarps), dim3(kProbeWarps * 32), 0, stream, s, k, skip_done);
}

// Called when a context is created, with its device current.
cudaError_t scan_kernel_setup() {
  return cudaFuncSetAttribute(scan_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kStreamSmemMax);
}

cudaError_t launch_scan(const Dev& s, int k, cudaStream_t stream) {
  // one CTA per tile while that keeps the device busy for one round; beyond that each CTA streams
  // through its share of its prompt's tiles
  const long long per_prompt = (long long)s.N * ((s.L + kScanTile - 1) / kScanTile);
  int set_slots = 64;
  while (set_slots < 4 * s.N) set_slots *= 2;
  const size_t dyn = ((size_t)4 * s.N + set_slots) * 4;
  if ((long long)s.G * per_prompt >= 148LL * 8 && (s.L & 3) == 0) {
    // streaming form: each CTA keeps kStreamStages tiles in flight
    constexpr int per_sm = 4;                                            // resident CTAs per SM (shared memory, registers)
    const size_t dyn_stream = dyn + (size_t)kStreamStages * kStreamTile * 4;
    const long long per_prompt_s = (long long)s.N * ((s.L + kStreamTile - 1) / kStreamTile);
    if (dyn_stream <= kStreamSmemMax) {
      // one round of resident CTAs while every CTA gets a few tiles only, four rounds for larger stores (set-ups then
      // overlap other CTAs' streaming)
      const long long tot = (long long)s.G * per_prompt > 148LL * 8 * 4 ? 148LL * per_sm * 4 : 148LL * per_sm;
      const long long ctas = std::max(1LL, std::min(per_prompt_s, tot / s.G));
      return launch_overlapped(scan_kernel<true>, dim3((unsigned)(ctas * s.G)), dim3(kStreamThreads), dyn_stream, stream, s,
                               k, (int)ctas, set_slots);
    }
  }
  const long long budget = 148LL * 8 * 4;
  long long ctas = per_prompt;
  if ((long long)s.G * per_prompt > budget) ctas = std::max(1LL, std::min(per_prompt, budget / s.G));
  return launch_overlapped(scan_kernel<false>, dim3((unsigned)(ctas * s.G)), dim3(kScanThreads), dyn, stream, s, k, (int)ctas,
                           set_slots);
}

cudaError_t launch_compact_matches(const Dev& s, int32_t* offsets, int32_t* gpos, size_t cap, cudaStream_t stream) {
  compact_matches_kernel<<<1, kProbeThreads, 0, stream>>>(s, offsets, gpos, cap);
  return cudaGetLastError();
}

}  // namespace sdms
